"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol that
include/ptq_linear.h declares, and its argument validation returns error codes (never aborts)."""
import ctypes
import os
import re

import numpy as np
import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    from paper_2412_20386_b200 import binding
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ptq_linear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ptq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert "ptq_linear_create" in names and "ptq_linear_forward" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings(lib):
    assert lib.ptq_status_string(0) == b"PTQ_OK"
    assert lib.ptq_status_string(8) == b"PTQ_ERR_TIMEOUT"
    assert lib.ptq_status_string(99) == b"PTQ_ERR_UNKNOWN"


def _create(lib, K, N, T, wq, dw, s, dx, bias=None, flags=0, out=True):
    h = ctypes.c_void_p()
    p = lambda a: None if a is None else a.ctypes.data_as(ctypes.c_void_p)
    st = lib.ptq_linear_create(ctypes.byref(h) if out else None, K, N, T, p(wq), p(dw), p(s), p(dx), p(bias), flags)
    return st, h


def test_create_rejects_bad_arguments_before_touching_a_device(lib):
    K, N, T = 16, 8, 4
    wq = np.ones((N, K), np.int8)
    dw = np.full(N, 0.01, np.float32)
    s = np.ones(K, np.float32)
    dx = np.ones(T, np.float32)
    assert _create(lib, K, N, T, wq, dw, s, dx, out=False)[0] == 1            # PTQ_ERR_NULL
    assert _create(lib, K, N, T, None, dw, s, dx)[0] == 1
    assert _create(lib, 0, N, T, wq, dw, s, dx)[0] == 2                       # PTQ_ERR_SHAPE
    assert _create(lib, 8193, N, T, wq, dw, s, dx)[0] == 2
    assert _create(lib, K, N, T, wq, dw, s, dx, flags=1)[0] == 3              # PTQ_ERR_VALUE
    for bad in (0.0, -1.0, np.inf, np.nan):
        s2 = s.copy(); s2[3] = bad
        assert _create(lib, K, N, T, wq, dw, s2, dx)[0] == 3
        dx2 = dx.copy(); dx2[1] = bad
        assert _create(lib, K, N, T, wq, dw, s, dx2)[0] == 3
        dw2 = dw.copy(); dw2[7] = bad
        assert _create(lib, K, N, T, wq, dw2, s, dx)[0] == 3
    w2 = wq.copy(); w2[5, 9] = -128
    st, _ = _create(lib, K, N, T, w2, dw, s, dx)
    assert st == 3 and b"-128" in lib.ptq_last_error()
    bias = np.zeros(N, np.float32); bias[0] = np.nan
    assert _create(lib, K, N, T, wq, dw, s, dx, bias)[0] == 3


def test_null_handles_are_refused_not_dereferenced(lib):
    assert lib.ptq_linear_workspace_bytes(None, 4, 0) == 0
    assert lib.ptq_linear_fused_supported(None) == 0
    assert lib.ptq_linear_gemm_variant(None, 1) == -1
    out = ctypes.c_double(-1.0)
    assert lib.ptq_probe(0, None, 0, 10, None, None) == 1                      # PTQ_ERR_NULL: no result pointer
    assert lib.ptq_probe(9, None, 0, 10, ctypes.byref(out), None) == 3         # PTQ_ERR_VALUE: unknown kind
    assert lib.ptq_probe(0, None, 0, 0, ctypes.byref(out), None) == 3          # iters out of range
    assert lib.ptq_probe(1, None, 1 << 20, 10, ctypes.byref(out), None) == 1   # a byte-moving kind needs a buffer
    assert out.value == 0.0
    assert lib.ptq_linear_forward(None, None, 1, None, None, 0, 0, None) == 1
    assert lib.ptq_quantize(None, None, 1, None, None) == 1
    assert lib.ptq_linear_device_status(None) == 1
    assert lib.ptq_calibrate(4, 4, 4, None, 1, None, None, None, None, None) == 1
    lib.ptq_linear_destroy(None)


def test_without_a_device_create_fails_with_an_error_code(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    K, N, T = 16, 8, 4
    st, h = _create(lib, K, N, T, np.ones((N, K), np.int8), np.full(N, 0.01, np.float32),
                    np.ones(K, np.float32), np.ones(T, np.float32))
    assert st in (5, 6) and not h.value        # PTQ_ERR_ARCH / PTQ_ERR_CUDA: loud, no fallback
