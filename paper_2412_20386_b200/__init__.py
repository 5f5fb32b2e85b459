"""B200-native PTS W8A8 linear layer (PTQ4VM, arXiv 2412.20386, Sec. 5.1).

The product is the C-ABI library declared in ``include/ptq_linear.h``; this
package holds its CUDA sources (``csrc/``), the build step (``build.py``), a thin
ctypes binding with the same entry points (``binding.py``) and the seeded
synthetic inputs (``workloads.py``).  The shared library is loaded on first use
and the binding raises if it is missing: there is no CPU fallback.
"""
from . import workloads  # noqa: F401
from .binding import (PtqError, PtqLinear, calibrate, calibrate_asym, calibrate_w4a4, search_act_step, library_path, load_library,  # noqa: F401
                      FLAG_FUSED_PROLOGUE, FLAG_CTA_PAIR)
