"""Build ``libptq_linear.so`` in-tree with nvcc for sm_100a.

    python -m paper_2412_20386_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  The CUDA runtime is linked statically and the
driver API is reached through the runtime's entry-point query, so the library
loads (and exports its symbols) on machines that have no NVIDIA driver.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_SO = os.path.join(_HERE, "libptq_linear.so")
_SOURCES = ["ptq_api.cu"]
_DEPS = ["ptq_api.cu", "ptq_gemm.cuh", "ptq_fused.cuh", "ptq_quantize.cuh", "ptq_quantize_dynamic.cuh",
         "ptq_calibrate.cuh", "ptq_probe.cuh", "ptx_sm100.cuh",
         os.path.join("..", "..", "include", "ptq_linear.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def up_to_date() -> bool:
    if not os.path.exists(_SO):
        return False
    t = os.path.getmtime(_SO)
    return all(os.path.getmtime(os.path.join(_CSRC, d)) <= t for d in _DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return _SO
    tmp = _SO + ".tmp.%d" % os.getpid()
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "static",
           "-Xptxas", "-v" if verbose else "-warn-spills"]
    cmd += [os.path.join(_CSRC, s) for s in _SOURCES]
    cmd += ["-o", tmp]
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout)
    if res.returncode != 0:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed (exit %d)" % res.returncode)
    os.replace(tmp, _SO)
    return _SO


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
