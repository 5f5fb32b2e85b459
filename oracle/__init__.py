"""ctypes binding of the CPU oracle (``ptq_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is the independent, slow CPU statement of
what the PTS W8A8 linear layer of PTQ4VM computes (Sec. 5.1, Eq. smooth_scale,
Eq. smooth).  Only the tests, the smoke check and the CPU-baseline leg of the
benchmark may import this package; the product package never does, and this
package imports nothing from the product.

Arrays are numpy: fp16 tensors travel as ``float16`` (viewed as ``uint16`` at
the C boundary), codes as ``int8``, accumulators as ``int32``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ptq_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libptq_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile ``ptq_oracle.c`` with gcc (no fast-math, no FMA contraction)."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    if (not force and os.path.exists(_SO)
            and os.path.getmtime(_SO) >= os.path.getmtime(_SRC)):
        return _SO
    tmp = _SO + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-std=c99", "-D_DEFAULT_SOURCE", "-Wall", "-shared", "-fPIC", _SRC,
           "-o", tmp, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _SO)
    return _SO


def _bind(path: str) -> ctypes.CDLL:
    L = ctypes.CDLL(path)
    c_long, c_int, vp = ctypes.c_long, ctypes.c_int, ctypes.c_void_p
    L.ptqo_num_threads.restype = c_int
    L.ptqo_half_to_float.restype = ctypes.c_float
    L.ptqo_half_to_float.argtypes = [ctypes.c_uint16]
    L.ptqo_double_to_half.restype = ctypes.c_uint16
    L.ptqo_double_to_half.argtypes = [ctypes.c_double]
    L.ptqo_quantize_one.restype = ctypes.c_int8
    L.ptqo_quantize_one.argtypes = [ctypes.c_uint16, ctypes.c_float, ctypes.c_float]
    L.ptqo_quantize.restype = None
    L.ptqo_quantize.argtypes = [vp, c_long, c_int, c_int, vp, vp, vp]
    L.ptqo_int_matmul.restype = c_int
    L.ptqo_int_matmul.argtypes = [vp, vp, c_long, c_int, c_int, vp]
    L.ptqo_dequant.restype = None
    L.ptqo_dequant.argtypes = [vp, c_long, c_int, c_int, vp, vp, vp, vp]
    L.ptqo_linear_forward_rows.restype = c_int
    L.ptqo_linear_forward_rows.argtypes = [vp, c_long, c_long, c_int, c_int, c_int,
                                           vp, vp, vp, vp, vp, vp, vp, vp]
    L.ptqo_calibrate.restype = None
    L.ptqo_calibrate.argtypes = [vp, c_int, c_int, c_int, vp, vp, c_int, vp, vp]
    L.ptqo_calibrate_per_tensor.restype = None
    L.ptqo_calibrate_per_tensor.argtypes = [vp, c_int, c_int, c_int, vp, vp, c_int, vp, vp]
    L.ptqo_quantize4_one.restype = ctypes.c_int8
    L.ptqo_quantize4_one.argtypes = [ctypes.c_uint16, ctypes.c_float, ctypes.c_float]
    L.ptqo_quantize4.restype = None
    L.ptqo_quantize4.argtypes = [vp, c_long, c_int, c_int, vp, vp, vp]
    L.ptqo_pack_int4.restype = None
    L.ptqo_pack_int4.argtypes = [vp, c_long, c_int, vp]
    L.ptqo_unpack_int4.restype = None
    L.ptqo_unpack_int4.argtypes = [vp, c_long, c_int, vp]
    L.ptqo_calibrate4.restype = None
    L.ptqo_calibrate4.argtypes = [vp, c_int, c_int, c_int, vp, vp, c_int, vp, vp]
    L.ptqo_search_act_step.restype = None
    L.ptqo_search_act_step.argtypes = [vp, c_int, c_int, c_int, vp, vp, c_int, c_int, vp, vp, vp]
    L.ptqo_quantize_dynamic.restype = None
    L.ptqo_quantize_dynamic.argtypes = [vp, c_long, c_int, vp, vp, vp]
    L.ptqo_quantize_asym_one.restype = ctypes.c_uint8
    L.ptqo_quantize_asym_one.argtypes = [ctypes.c_uint16, ctypes.c_float, ctypes.c_float, c_int]
    L.ptqo_quantize_asym.restype = None
    L.ptqo_quantize_asym.argtypes = [vp, c_long, c_int, c_int, vp, vp, vp, vp]
    L.ptqo_int_matmul_asym.restype = c_int
    L.ptqo_int_matmul_asym.argtypes = [vp, vp, c_int, vp, c_long, c_int, c_int, vp]
    L.ptqo_calibrate_asym.restype = None
    L.ptqo_calibrate_asym.argtypes = [vp, c_int, c_int, c_int, vp, vp, c_int, vp, vp, vp]
    L.ptqo_linear_forward_rows_asym.restype = c_int
    L.ptqo_linear_forward_rows_asym.argtypes = [vp, c_long, c_long, c_int, c_int, c_int,
                                                vp, vp, vp, vp, vp, vp, vp, vp, vp]
    return L


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


class use_library:
    """Context manager for the tests of the tests: run the oracle's Python API against another build of
    ``ptq_oracle.c`` (a copy with a planted mistake) to show that the pins notice it."""

    def __init__(self, source_text: str, workdir: str):
        self.src = os.path.join(workdir, "ptq_oracle_mutant.c")
        self.so = os.path.join(workdir, "libptq_oracle_mutant_%d.so" % (abs(hash(source_text)) % 10 ** 9))
        with open(self.src, "w") as f:
            f.write(source_text)
        subprocess.run(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-std=c99",
                        "-D_DEFAULT_SOURCE", "-shared", "-fPIC", self.src, "-o", self.so, "-lm"], check=True)

    def __enter__(self):
        global _lib
        self.saved = lib()
        _lib = _bind(self.so)
        return self

    def __exit__(self, *exc):
        global _lib
        _lib = self.saved
        return False


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError("expected %s, got %s" % (np.dtype(dtype), a.dtype))
    return a


def num_threads() -> int:
    return int(lib().ptqo_num_threads())


def half_to_float(bits: int) -> float:
    return float(lib().ptqo_half_to_float(int(bits)))


def double_to_half_bits(v: float) -> int:
    return int(lib().ptqo_double_to_half(float(v)))


def quantize_one(x_bits: int, s: float, dx: float) -> int:
    return int(lib().ptqo_quantize_one(int(x_bits), float(s), float(dx)))


def quantize(x, T, s, dx):
    """Q1: x fp16 [M,K] -> int8 codes [M,K]; s fp32 [K]; dx fp32 [T]."""
    x = _c(x, np.float16)
    M, K = x.shape
    s = _c(s, np.float32)
    dx = _c(dx, np.float32)
    assert s.shape == (K,) and dx.shape == (T,)
    q = np.empty((M, K), np.int8)
    lib().ptqo_quantize(_p(x), M, K, T, _p(s), _p(dx), _p(q))
    return q


def int_matmul(q, wq):
    """G1: q int8 [M,K] x wq int8 [N,K]^T -> int32 [M,N] (raises on int32 overflow)."""
    q = _c(q, np.int8)
    wq = _c(wq, np.int8)
    M, K = q.shape
    N, K2 = wq.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    if lib().ptqo_int_matmul(_p(q), _p(wq), M, K, N, _p(acc)):
        raise OverflowError("accumulator does not fit in int32")
    return acc


def dequant(acc, T, dx, dw, bias=None):
    """E1: int32 [M,N] -> fp16 [M,N] = acc * dx[m mod T] * dw[n] (+ bias[n])."""
    acc = _c(acc, np.int32)
    M, N = acc.shape
    dx = _c(dx, np.float32)
    dw = _c(dw, np.float32)
    if bias is not None:
        bias = _c(bias, np.float32)
        assert bias.shape == (N,)
    assert dx.shape == (T,) and dw.shape == (N,)
    y = np.empty((M, N), np.float16)
    lib().ptqo_dequant(_p(acc), M, N, T, _p(dx), _p(dw), _p(bias), _p(y))
    return y


def linear_forward(x, T, wq, dw, s, dx, bias=None, rows=None, taps=False):
    """Whole path Q1 -> G1 -> E1 on rows [m0, m1) of x fp16 [M,K].

    Returns y fp16 [m1-m0, N], or (y, q, acc) when ``taps`` is set.
    """
    x = _c(x, np.float16)
    M, K = x.shape
    wq = _c(wq, np.int8)
    N = wq.shape[0]
    assert wq.shape == (N, K)
    dw = _c(dw, np.float32)
    s = _c(s, np.float32)
    dx = _c(dx, np.float32)
    assert dw.shape == (N,) and s.shape == (K,) and dx.shape == (T,)
    if bias is not None:
        bias = _c(bias, np.float32)
        assert bias.shape == (N,)
    m0, m1 = (0, M) if rows is None else rows
    assert 0 <= m0 <= m1 <= M
    R = m1 - m0
    y = np.empty((R, N), np.float16)
    q = np.empty((R, K), np.int8) if taps else None
    acc = np.empty((R, N), np.int32) if taps else None
    rc = lib().ptqo_linear_forward_rows(_p(x), m0, m1, K, N, T, _p(wq), _p(dw), _p(s),
                                        _p(dx), _p(bias), _p(y), _p(q), _p(acc))
    if rc < 0:
        raise ValueError("K too large for the oracle's row buffer")
    if rc:
        raise OverflowError("accumulator does not fit in int32")
    return (y, q, acc) if taps else y


def calibrate(xcal, wq, dw):
    """Q0: xcal fp16 [Bc,T,K], wq int8 [N,K], dw fp32 [N] -> (s fp32 [K], dx fp32 [T])."""
    xcal = _c(xcal, np.float16)
    Bc, T, K = xcal.shape
    wq = _c(wq, np.int8)
    N = wq.shape[0]
    assert wq.shape == (N, K)
    dw = _c(dw, np.float32)
    s = np.empty(K, np.float32)
    dx = np.empty(T, np.float32)
    lib().ptqo_calibrate(_p(xcal), Bc, T, K, _p(wq), _p(dw), N, _p(s), _p(dx))
    return s, dx


def calibrate_per_tensor(xcal, wq, dw):
    """Per-tensor static comparator: (s fp32 [K], delta) with ONE activation step for all token positions."""
    xcal = _c(xcal, np.float16)
    Bc, T, K = xcal.shape
    wq = _c(wq, np.int8)
    N = wq.shape[0]
    assert wq.shape == (N, K)
    dw = _c(dw, np.float32)
    s = np.empty(K, np.float32)
    delta = np.empty(1, np.float32)
    lib().ptqo_calibrate_per_tensor(_p(xcal), Bc, T, K, _p(wq), _p(dw), N, _p(s), _p(delta))
    return s, np.float32(delta[0])


# --------------------------------------------------------------------------- #
# asymmetric PTS (step and zero offset per token position)                     #
# --------------------------------------------------------------------------- #
def quantize_asym_one(x_bits: int, s: float, dx: float, z: int) -> int:
    return int(lib().ptqo_quantize_asym_one(int(x_bits), float(s), float(dx), int(z)))


def quantize_asym(x, T, s, dx, z):
    """x fp16 [M,K] -> uint8 codes [M,K] = clip(round((x/s)/dx[t]) + z[t], 0, 255)."""
    x = _c(x, np.float16)
    M, K = x.shape
    s = _c(s, np.float32)
    dx = _c(dx, np.float32)
    z = _c(z, np.int32)
    assert s.shape == (K,) and dx.shape == (T,) and z.shape == (T,)
    c = np.empty((M, K), np.uint8)
    lib().ptqo_quantize_asym(_p(x), M, K, T, _p(s), _p(dx), _p(z), _p(c))
    return c


def int_matmul_asym(c, z, T, wq):
    """acc[m,n] = sum_k (c[m,k] - z[m mod T]) * wq[n,k] (raises on int32 overflow)."""
    c = _c(c, np.uint8)
    z = _c(z, np.int32)
    wq = _c(wq, np.int8)
    M, K = c.shape
    N = wq.shape[0]
    assert wq.shape == (N, K) and z.shape == (T,)
    acc = np.empty((M, N), np.int32)
    if lib().ptqo_int_matmul_asym(_p(c), _p(z), T, _p(wq), M, K, N, _p(acc)):
        raise OverflowError("accumulator does not fit in int32")
    return acc


def calibrate_asym(xcal, wq, dw):
    """xcal fp16 [Bc,T,K] -> (s fp32 [K], dx fp32 [T], z int32 [T])."""
    xcal = _c(xcal, np.float16)
    Bc, T, K = xcal.shape
    wq = _c(wq, np.int8)
    N = wq.shape[0]
    assert wq.shape == (N, K)
    dw = _c(dw, np.float32)
    s = np.empty(K, np.float32)
    dx = np.empty(T, np.float32)
    z = np.empty(T, np.int32)
    lib().ptqo_calibrate_asym(_p(xcal), Bc, T, K, _p(wq), _p(dw), N, _p(s), _p(dx), _p(z))
    return s, dx, z


def linear_forward_asym(x, T, wq, dw, s, dx, z, bias=None, rows=None, taps=False):
    """Whole asymmetric path on rows [m0, m1): y fp16, or (y, codes uint8, acc int32) with taps."""
    x = _c(x, np.float16)
    M, K = x.shape
    wq = _c(wq, np.int8)
    N = wq.shape[0]
    assert wq.shape == (N, K)
    dw = _c(dw, np.float32)
    s = _c(s, np.float32)
    dx = _c(dx, np.float32)
    z = _c(z, np.int32)
    assert dw.shape == (N,) and s.shape == (K,) and dx.shape == (T,) and z.shape == (T,)
    if bias is not None:
        bias = _c(bias, np.float32)
    m0, m1 = (0, M) if rows is None else rows
    R = m1 - m0
    y = np.empty((R, N), np.float16)
    c = np.empty((R, K), np.uint8) if taps else None
    acc = np.empty((R, N), np.int32) if taps else None
    rc = lib().ptqo_linear_forward_rows_asym(_p(x), m0, m1, K, N, T, _p(wq), _p(dw), _p(s), _p(dx), _p(z),
                                             _p(bias), _p(y), _p(c), _p(acc))
    if rc < 0:
        raise ValueError("K too large for the oracle's row buffer")
    if rc:
        raise OverflowError("accumulator does not fit in int32")
    return (y, c, acc) if taps else y


# --------------------------------------------------------------------------- #
# comparator: per-token dynamic quantization                                   #
# --------------------------------------------------------------------------- #
def quantize_dynamic(x, s):
    """x fp16 [M,K] -> (int8 codes [M,K], per-row steps fp32 [M]) with dx_row = max|x/s| / 127 per row."""
    x = _c(x, np.float16)
    M, K = x.shape
    s = _c(s, np.float32)
    assert s.shape == (K,)
    q = np.empty((M, K), np.int8)
    dx_row = np.empty(M, np.float32)
    lib().ptqo_quantize_dynamic(_p(x), M, K, _p(s), _p(q), _p(dx_row))
    return q, dx_row


def linear_forward_dynamic(x, wq, dw, s, bias=None, taps=False):
    """Dynamic comparator end to end: codes and row steps, contraction, dequantization with T = M."""
    q, dx_row = quantize_dynamic(x, s)
    acc = int_matmul(q, wq)
    y = dequant(acc, q.shape[0], dx_row, dw, bias)
    return (y, q, acc, dx_row) if taps else y


# --------------------------------------------------------------------------- #
# step-size search (Sec. 5.2, second stage)                                    #
# --------------------------------------------------------------------------- #
def search_act_step(xcal, s, base, n_grid=100, j_lo=20):
    """xcal fp16 [Bc,T,K] -> (dx fp32 [T], best int32 [T], loss fp64 [T, n_grid-j_lo+1]):
    per token position the candidate base[t]*j/n_grid (j_lo <= j <= n_grid) of least squared error."""
    xcal = _c(xcal, np.float16)
    Bc, T, K = xcal.shape
    s = _c(s, np.float32)
    base = _c(base, np.float32)
    assert s.shape == (K,) and base.shape == (T,) and 1 <= j_lo <= n_grid
    C = n_grid - j_lo + 1
    loss = np.empty((T, C), np.float64)
    best = np.empty(T, np.int32)
    dx = np.empty(T, np.float32)
    lib().ptqo_search_act_step(_p(xcal), Bc, T, K, _p(s), _p(base), n_grid, j_lo, _p(loss), _p(best), _p(dx))
    return dx, best, loss


# --------------------------------------------------------------------------- #
# 4-bit variant (W4A4): signed range [-8, 7], two values per byte              #
# --------------------------------------------------------------------------- #
def quantize4_one(x_bits: int, s: float, dx: float) -> int:
    return int(lib().ptqo_quantize4_one(int(x_bits), float(s), float(dx)))


def quantize4(x, T, s, dx):
    """x fp16 [M,K] -> int8-held 4-bit codes [M,K] = clip(round((x/s)/dx[t]), -8, 7)."""
    x = _c(x, np.float16)
    M, K = x.shape
    s = _c(s, np.float32)
    dx = _c(dx, np.float32)
    assert s.shape == (K,) and dx.shape == (T,)
    q = np.empty((M, K), np.int8)
    lib().ptqo_quantize4(_p(x), M, K, T, _p(s), _p(dx), _p(q))
    return q


def pack_int4(d):
    """int8 [rows, cols] with values in [-8, 7] -> uint8 [rows, (cols+1)//2], low nibble = even index."""
    d = _c(d, np.int8)
    rows, cols = d.shape
    out = np.empty((rows, (cols + 1) // 2), np.uint8)
    lib().ptqo_pack_int4(_p(d), rows, cols, _p(out))
    return out


def unpack_int4(packed, cols):
    packed = _c(packed, np.uint8)
    rows = packed.shape[0]
    assert packed.shape[1] == (cols + 1) // 2
    out = np.empty((rows, cols), np.int8)
    lib().ptqo_unpack_int4(_p(packed), rows, cols, _p(out))
    return out


def calibrate4(xcal, wq, dw):
    """Min-max calibration for 4-bit activations: (s fp32 [K], dx fp32 [T]) with dx = max|x/s| / 7."""
    xcal = _c(xcal, np.float16)
    Bc, T, K = xcal.shape
    wq = _c(wq, np.int8)
    N = wq.shape[0]
    assert wq.shape == (N, K)
    dw = _c(dw, np.float32)
    s = np.empty(K, np.float32)
    dx = np.empty(T, np.float32)
    lib().ptqo_calibrate4(_p(xcal), Bc, T, K, _p(wq), _p(dw), N, _p(s), _p(dx))
    return s, dx


def linear_forward4(x, T, wq4, dw, s, dx, bias=None, taps=False):
    """W4A4 end to end: 4-bit codes, contraction with the 4-bit weights (held one per int8), dequantization."""
    x = _c(x, np.float16)
    q = quantize4(x, T, s, dx)
    acc = int_matmul(q, wq4)
    y = dequant(acc, T, dx, dw, bias)
    return (y, q, acc) if taps else y
