"""ctypes binding of ``libptq_linear.so`` (the C ABI of ``include/ptq_linear.h``).

Argument marshalling only: every step of the path (quantize, integer GEMM,
dequantize, calibration reductions) runs in the library's CUDA kernels.  torch
tensors are used for device memory and streams; their ``data_ptr()`` crosses
the boundary as a plain pointer.  There is no fallback: if the library is
missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libptq_linear.so")

FLAG_NONE = 0
FLAG_FUSED_PROLOGUE = 1
FLAG_CTA_PAIR = 2
STATIC_SCRATCH_BYTES = 32 * 1024 * 1024

_STATUS_NAMES = {0: "PTQ_OK", 1: "PTQ_ERR_NULL", 2: "PTQ_ERR_SHAPE", 3: "PTQ_ERR_VALUE",
                 4: "PTQ_ERR_ALIGN", 5: "PTQ_ERR_ARCH", 6: "PTQ_ERR_CUDA", 7: "PTQ_ERR_NOMEM",
                 8: "PTQ_ERR_TIMEOUT"}

_lib = None


class PtqError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__("%s: %s" % (_STATUS_NAMES.get(status, status), text))
        self.status = status


def library_path() -> str:
    return _SO


def load_library() -> ctypes.CDLL:
    """Load the shared library (built by ``paper_2412_20386_b200.build``); raise if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_SO):
        raise ImportError(
            "%s not found: build it with `python -m paper_2412_20386_b200.build` "
            "(nvcc, sm_100a). There is no fallback implementation." % _SO)
    L = ctypes.CDLL(_SO)
    vp, ci, cu, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint, ctypes.c_size_t
    L.ptq_linear_create.restype = ci
    L.ptq_linear_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, vp, vp, vp, vp, vp, cu]
    L.ptq_linear_create_asym.restype = ci
    L.ptq_linear_create_asym.argtypes = [ctypes.POINTER(vp), ci, ci, ci, vp, vp, vp, vp, vp, vp, cu]
    L.ptq_calibrate_asym.restype = ci
    L.ptq_calibrate_asym.argtypes = [ci, ci, ci, vp, ci, vp, vp, vp, vp, vp, vp]
    L.ptq_linear_destroy.restype = None
    L.ptq_linear_destroy.argtypes = [vp]
    L.ptq_linear_workspace_bytes.restype = sz
    L.ptq_linear_workspace_bytes.argtypes = [vp, ci, cu]
    L.ptq_linear_forward.restype = ci
    L.ptq_linear_forward.argtypes = [vp, vp, ci, vp, vp, sz, cu, vp]
    L.ptq_probe.restype = ci
    L.ptq_probe.argtypes = [ci, vp, sz, ci, ctypes.POINTER(ctypes.c_double), vp]
    L.ptq_linear_gemm_variant.restype = ci
    L.ptq_linear_gemm_variant.argtypes = [vp, ci]
    L.ptq_linear_forward_static.restype = ci
    L.ptq_linear_forward_static.argtypes = [vp, vp, ci, vp, vp]
    L.ptq_linear_workspace_bytes_dynamic.restype = sz
    L.ptq_linear_workspace_bytes_dynamic.argtypes = [vp, ci]
    L.ptq_linear_forward_dynamic.restype = ci
    L.ptq_linear_forward_dynamic.argtypes = [vp, vp, ci, vp, vp, sz, vp]
    L.ptq_linear_forward_dynamic_debug.restype = ci
    L.ptq_linear_forward_dynamic_debug.argtypes = [vp, vp, ci, vp, vp, vp, vp, vp, sz, vp]
    L.ptq_linear_fused_supported.restype = ci
    L.ptq_linear_fused_supported.argtypes = [vp]
    L.ptq_quantize.restype = ci
    L.ptq_quantize.argtypes = [vp, vp, ci, vp, vp]
    L.ptq_linear_gemm_dequant.restype = ci
    L.ptq_linear_gemm_dequant.argtypes = [vp, vp, ci, vp, vp]
    L.ptq_linear_code_pitch.restype = ci
    L.ptq_linear_code_pitch.argtypes = [vp]
    L.ptq_linear_forward_debug.restype = ci
    L.ptq_linear_forward_debug.argtypes = [vp, vp, ci, vp, vp, vp, vp, sz, cu, vp]
    L.ptq_calibrate.restype = ci
    L.ptq_calibrate.argtypes = [ci, ci, ci, vp, ci, vp, vp, vp, vp, vp]
    L.ptq_linear_create_w4a4.restype = ci
    L.ptq_linear_create_w4a4.argtypes = [ctypes.POINTER(vp), ci, ci, ci, vp, vp, vp, vp, vp, cu]
    L.ptq_linear_selftest_wait_timeout.restype = ci
    L.ptq_linear_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint, vp, vp]
    L.ptq_calibrate_per_tensor.restype = ci
    L.ptq_calibrate_per_tensor.argtypes = [ci, ci, ci, vp, ci, vp, vp, vp, vp, vp]
    L.ptq_calibrate_w4a4.restype = ci
    L.ptq_calibrate_w4a4.argtypes = [ci, ci, ci, vp, ci, vp, vp, vp, vp, vp]
    L.ptq_quantize_packed4.restype = ci
    L.ptq_quantize_packed4.argtypes = [vp, vp, ci, vp, vp, sz, vp]
    L.ptq_search_act_step.restype = ci
    L.ptq_search_act_step.argtypes = [ci, ci, vp, ci, vp, vp, ci, ci, vp, vp, vp, vp]
    L.ptq_linear_describe.restype = ci
    L.ptq_linear_describe.argtypes = [vp, ctypes.c_char_p, ci]
    L.ptq_linear_device_status.restype = ci
    L.ptq_linear_device_status.argtypes = [vp]
    L.ptq_kernel_launch_count.restype = ctypes.c_ulonglong
    L.ptq_kernel_launch_count.argtypes = []
    L.ptq_status_string.restype = ctypes.c_char_p
    L.ptq_status_string.argtypes = [ci]
    L.ptq_last_error.restype = ctypes.c_char_p
    L.ptq_last_error.argtypes = []
    _lib = L
    return L


def _check(status: int):
    if status != 0:
        raise PtqError(status, load_library().ptq_last_error().decode("utf-8", "replace"))


def _host(a, dtype, shape=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=dtype)
    if shape is not None and a.shape != tuple(shape):
        raise ValueError("expected shape %s, got %s" % (tuple(shape), a.shape))
    return a


def _hp(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(int(stream.cuda_stream))


def _scratch(nbytes: int, device, stream):
    """A temporary device buffer for one call.  The kernels run on `stream`, which need not be the
    stream torch's allocator associates the block with: recording the use keeps the block from being
    handed out again while the kernels still read it."""
    import torch
    buf = torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)
    if stream is not None:
        buf.record_stream(stream)
    return buf


def kernel_launch_count() -> int:
    return int(load_library().ptq_kernel_launch_count())


PROBE_STORE16, PROBE_TMA_STORE, PROBE_OPERAND_PULL, PROBE_LAUNCH, PROBE_LAUNCH_PDL = 0, 1, 2, 3, 4


def probe(kind: int, buf=None, iters: int = 20, stream=None) -> float:
    """``ptq_probe``: GB/s (kinds 0-2, over the device uint8 tensor ``buf``) or microseconds per launch (kinds 3-4)."""
    L = load_library()
    out = ctypes.c_double(0.0)
    ptr, nbytes = (None, 0) if buf is None else (buf.data_ptr(), buf.numel() * buf.element_size())
    _check(L.ptq_probe(int(kind), ptr, nbytes, int(iters), ctypes.byref(out), _stream_ptr(stream)))
    return float(out.value)


class PtqLinear:
    """One PTS W8A8 linear layer on the current CUDA device (``ptq_linear_create``)."""

    def __init__(self, w_q, w_step, smooth, act_step, bias=None, flags: int = 0, act_zero=None, packed4_K=None):
        L = load_library()
        self.w4a4 = packed4_K is not None
        if self.w4a4:                                            # ``ptq_linear_create_w4a4``: w_q is [N, (K+1)//2] bytes
            w_q = _host(w_q, np.uint8)
            if w_q.ndim != 2 or w_q.shape[1] != (int(packed4_K) + 1) // 2:
                raise ValueError("packed w_q must be [N, (K+1)//2] bytes")
            self.N, self.K = int(w_q.shape[0]), int(packed4_K)
        else:
            w_q = _host(w_q, np.int8)
            if w_q.ndim != 2:
                raise ValueError("w_q must be [N,K]")
            self.N, self.K = int(w_q.shape[0]), int(w_q.shape[1])
        act_step = _host(act_step, np.float32)
        self.T = int(act_step.shape[0])
        w_step = _host(w_step, np.float32, (self.N,))
        smooth = _host(smooth, np.float32, (self.K,))
        bias = _host(bias, np.float32, (self.N,))
        h = ctypes.c_void_p()
        self.asym = act_zero is not None
        if self.w4a4:
            if self.asym:
                raise ValueError("W4A4 layers are symmetric")
            _check(L.ptq_linear_create_w4a4(ctypes.byref(h), self.K, self.N, self.T, _hp(w_q), _hp(w_step),
                                            _hp(smooth), _hp(act_step), _hp(bias), flags))
        elif self.asym:                                          # ``ptq_linear_create_asym``: unsigned codes
            act_zero = _host(act_zero, np.int32, (self.T,))
            _check(L.ptq_linear_create_asym(ctypes.byref(h), self.K, self.N, self.T, _hp(w_q), _hp(w_step),
                                            _hp(smooth), _hp(act_step), _hp(act_zero), _hp(bias), flags))
        else:
            _check(L.ptq_linear_create(ctypes.byref(h), self.K, self.N, self.T, _hp(w_q), _hp(w_step),
                                       _hp(smooth), _hp(act_step), _hp(bias), flags))
        self._h = h
        self._L = L

    def close(self):
        if getattr(self, "_h", None):
            self._L.ptq_linear_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- queries ---------------------------------------------------------------
    def workspace_bytes(self, B: int, flags: int = 0) -> int:
        return int(self._L.ptq_linear_workspace_bytes(self._h, int(B), flags))

    def fused_supported(self) -> bool:
        return bool(self._L.ptq_linear_fused_supported(self._h))

    def describe(self) -> str:
        buf = ctypes.create_string_buffer(512)
        self._L.ptq_linear_describe(self._h, buf, 512)
        return buf.value.decode()

    def device_status(self):
        _check(self._L.ptq_linear_device_status(self._h))

    def selftest_wait_timeout(self, limit_us: int = 50, stream=None):
        """``ptq_linear_selftest_wait_timeout``: returns (short wait result, long wait result, ns waited)."""
        out = (ctypes.c_uint * 3)()
        _check(self._L.ptq_linear_selftest_wait_timeout(self._h, int(limit_us), out, _stream_ptr(stream)))
        return int(out[0]), int(out[1]), int(out[2])

    # -- calls -----------------------------------------------------------------
    def _batch(self, x):
        import torch
        if x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
            raise ValueError("x must be a contiguous CUDA float16 tensor")
        if x.numel() % (self.T * self.K) != 0 or x.shape[-1] != self.K:
            raise ValueError("x must be [B,T,K] with T=%d K=%d" % (self.T, self.K))
        return x.numel() // (self.T * self.K)

    def forward(self, x, y=None, workspace=None, flags: int = 0, stream=None):
        """``ptq_linear_forward``: x fp16 [B,T,K] -> y fp16 [B,T,N] (both on the device)."""
        import torch
        B = self._batch(x)
        if y is None:
            y = torch.empty((B, self.T, self.N), dtype=torch.float16, device=x.device)
        if flags & FLAG_FUSED_PROLOGUE and x.data_ptr() % 16:
            need = self.workspace_bytes(B, 0)      # an x that is not 16-byte aligned takes the two-kernel path
        else:
            need = self.workspace_bytes(B, flags)
        if workspace is None and need:
            workspace = _scratch(need, x.device, stream)
        wptr = workspace.data_ptr() if workspace is not None else None
        wbytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
        _check(self._L.ptq_linear_forward(self._h, x.data_ptr(), B, y.data_ptr(), wptr, wbytes,
                                          flags, _stream_ptr(stream)))
        return y

    def forward_static(self, x, y, stream=None):
        """``ptq_linear_forward_static``: forward pass that allocates nothing.

        The caller passes both x and y; the int8 codes go to the scratch array built into the
        library (at most ``STATIC_SCRATCH_BYTES``), which all calls on a device share.
        """
        B = self._batch(x)
        if tuple(y.shape) != (B, self.T, self.N) or y.dtype != x.dtype or not y.is_contiguous() or not y.is_cuda:
            raise ValueError("y must be a contiguous CUDA float16 tensor [B,T,N]")
        _check(self._L.ptq_linear_forward_static(self._h, x.data_ptr(), B, y.data_ptr(), _stream_ptr(stream)))
        return y

    def workspace_bytes_dynamic(self, B: int) -> int:
        return int(self._L.ptq_linear_workspace_bytes_dynamic(self._h, B))

    def forward_dynamic(self, x, y=None, workspace=None, stream=None):
        """``ptq_linear_forward_dynamic``: the per-token dynamic comparator (row steps measured at run time)."""
        import torch
        B = self._batch(x)
        if y is None:
            y = torch.empty((B, self.T, self.N), dtype=torch.float16, device=x.device)
        if workspace is None:
            workspace = _scratch(self.workspace_bytes_dynamic(B), x.device, stream)
        _check(self._L.ptq_linear_forward_dynamic(self._h, x.data_ptr(), B, y.data_ptr(), workspace.data_ptr(),
                                                  workspace.numel() * workspace.element_size(),
                                                  _stream_ptr(stream)))
        return y

    def forward_dynamic_debug(self, x, stream=None):
        """``ptq_linear_forward_dynamic_debug``: returns (y, q int8 [B,T,K], acc int32 [B,T,N], step fp32 [B*T])."""
        import torch
        B = self._batch(x)
        dev = x.device
        y = torch.empty((B, self.T, self.N), dtype=torch.float16, device=dev)
        q = torch.empty((B, self.T, self.K), dtype=torch.int8, device=dev)
        acc = torch.empty((B, self.T, self.N), dtype=torch.int32, device=dev)
        step = torch.empty(B * self.T, dtype=torch.float32, device=dev)
        need = self.workspace_bytes_dynamic(B)
        ws = _scratch(need, dev, stream)
        _check(self._L.ptq_linear_forward_dynamic_debug(self._h, x.data_ptr(), B, y.data_ptr(), q.data_ptr(),
                                                        acc.data_ptr(), step.data_ptr(), ws.data_ptr(), need,
                                                        _stream_ptr(stream)))
        return y, q, acc, step

    def quantize(self, x, q=None, stream=None):
        """``ptq_quantize``: x fp16 [B,T,K] -> int8 codes [B,T,K]."""
        import torch
        B = self._batch(x)
        if q is None:
            q = torch.empty((B, self.T, self.K), dtype=torch.uint8 if self.asym else torch.int8, device=x.device)
        _check(self._L.ptq_quantize(self._h, x.data_ptr(), B, q.data_ptr(), _stream_ptr(stream)))
        return q

    def quantize_packed4(self, x, stream=None):
        """``ptq_quantize_packed4``: x fp16 [B,T,K] -> 4-bit codes packed two per byte, uint8 [B,T,(K+1)//2]."""
        import torch
        B = self._batch(x)
        out = torch.empty((B, self.T, (self.K + 1) // 2), dtype=torch.uint8, device=x.device)
        need = self.workspace_bytes(B, 0)
        ws = _scratch(need, x.device, stream)
        _check(self._L.ptq_quantize_packed4(self._h, x.data_ptr(), B, out.data_ptr(), ws.data_ptr(), need,
                                            _stream_ptr(stream)))
        return out

    def code_pitch(self) -> int:
        return int(self._L.ptq_linear_code_pitch(self._h))

    def gemm_variant(self, B: int) -> int:
        """``ptq_linear_gemm_variant``: 0 streaming kernel, 1 streaming with two epilogue teams, 2 panel kernel."""
        return int(self._L.ptq_linear_gemm_variant(self._h, int(B)))

    def gemm_dequant(self, q, B: int, y=None, stream=None):
        """``ptq_linear_gemm_dequant``: int8 codes [B*T, code_pitch()] -> y fp16 [B,T,N]."""
        import torch
        if q.dtype not in (torch.int8, torch.uint8) or not q.is_cuda or not q.is_contiguous():
            raise ValueError("q must be a contiguous CUDA int8 tensor")
        if q.numel() < B * self.T * self.code_pitch():
            raise ValueError("q holds fewer than B*T rows of code_pitch() bytes")
        if y is None:
            y = torch.empty((B, self.T, self.N), dtype=torch.float16, device=q.device)
        _check(self._L.ptq_linear_gemm_dequant(self._h, q.data_ptr(), int(B), y.data_ptr(), _stream_ptr(stream)))
        return y

    def forward_debug(self, x, flags: int = 0, want_q=True, want_acc=True, stream=None):
        """``ptq_linear_forward_debug``: returns (y, q or None, acc or None)."""
        import torch
        B = self._batch(x)
        dev = x.device
        y = torch.empty((B, self.T, self.N), dtype=torch.float16, device=dev)
        q = torch.empty((B, self.T, self.K), dtype=torch.uint8 if self.asym else torch.int8,
                        device=dev) if want_q else None
        acc = torch.empty((B, self.T, self.N), dtype=torch.int32, device=dev) if want_acc else None
        need = self.workspace_bytes(B, 0)
        ws = _scratch(need, dev, stream)
        _check(self._L.ptq_linear_forward_debug(
            self._h, x.data_ptr(), B, y.data_ptr(),
            q.data_ptr() if q is not None else None,
            acc.data_ptr() if acc is not None else None,
            ws.data_ptr(), need, flags, _stream_ptr(stream)))
        return y, q, acc


def calibrate(xcal, w_q, w_step, stream=None, per_tensor: bool = False):
    """``ptq_calibrate``: device fp16 [Bc,T,K] -> (s fp32 [K], dx fp32 [T]) as numpy arrays.
    ``per_tensor=True`` calls ``ptq_calibrate_per_tensor`` (one step, repeated T times)."""
    import torch
    L = load_library()
    if xcal.dtype != torch.float16 or not xcal.is_cuda or not xcal.is_contiguous() or xcal.dim() != 3:
        raise ValueError("xcal must be a contiguous CUDA float16 tensor [Bc,T,K]")
    Bc, T, K = (int(v) for v in xcal.shape)
    w_q = _host(w_q, np.int8)
    N = int(w_q.shape[0])
    if w_q.shape != (N, K):
        raise ValueError("w_q must be [N,K]")
    w_step = _host(w_step, np.float32, (N,))
    s = np.empty(K, np.float32)
    dx = np.empty(T, np.float32)
    fn = L.ptq_calibrate_per_tensor if per_tensor else L.ptq_calibrate
    _check(fn(K, N, T, xcal.data_ptr(), Bc, _hp(w_q), _hp(w_step), _hp(s), _hp(dx), _stream_ptr(stream)))
    return s, dx


def calibrate_asym(xcal, w_q, w_step, stream=None):
    """``ptq_calibrate_asym``: device fp16 [Bc,T,K] -> (s fp32 [K], dx fp32 [T], z int32 [T])."""
    import torch
    L = load_library()
    if xcal.dtype != torch.float16 or not xcal.is_cuda or not xcal.is_contiguous() or xcal.dim() != 3:
        raise ValueError("xcal must be a contiguous CUDA float16 tensor [Bc,T,K]")
    Bc, T, K = (int(v) for v in xcal.shape)
    w_q = _host(w_q, np.int8)
    N = int(w_q.shape[0])
    if w_q.shape != (N, K):
        raise ValueError("w_q must be [N,K]")
    w_step = _host(w_step, np.float32, (N,))
    s = np.empty(K, np.float32)
    dx = np.empty(T, np.float32)
    z = np.empty(T, np.int32)
    _check(L.ptq_calibrate_asym(K, N, T, xcal.data_ptr(), Bc, _hp(w_q), _hp(w_step), _hp(s), _hp(dx), _hp(z),
                                _stream_ptr(stream)))
    return s, dx, z


def search_act_step(xcal, smooth, base_step, n_grid: int = 100, j_lo: int = 20, want_loss: bool = False, stream=None):
    """``ptq_search_act_step``: device fp16 [Bc,T,K] -> (dx fp32 [T], best j int32 [T], loss fp64 [T,C] or None)."""
    import torch
    L = load_library()
    if xcal.dtype != torch.float16 or not xcal.is_cuda or not xcal.is_contiguous() or xcal.dim() != 3:
        raise ValueError("xcal must be a contiguous CUDA float16 tensor [Bc,T,K]")
    Bc, T, K = (int(v) for v in xcal.shape)
    smooth = _host(smooth, np.float32, (K,))
    base_step = _host(base_step, np.float32, (T,))
    dx = np.empty(T, np.float32)
    best = np.empty(T, np.int32)
    loss = np.empty((T, max(n_grid - j_lo + 1, 1)), np.float64) if want_loss else None
    _check(L.ptq_search_act_step(K, T, xcal.data_ptr(), Bc, smooth.ctypes.data, base_step.ctypes.data, n_grid, j_lo,
                                 dx.ctypes.data, best.ctypes.data,
                                 loss.ctypes.data if loss is not None else None, _stream_ptr(stream)))
    return dx, best, loss


def calibrate_w4a4(xcal, w_q_packed, K: int, w_step, stream=None):
    """``ptq_calibrate_w4a4``: device fp16 [Bc,T,K], packed 4-bit weights -> (s fp32 [K], dx fp32 [T] = max|x/s|/7)."""
    import torch
    L = load_library()
    if xcal.dtype != torch.float16 or not xcal.is_cuda or not xcal.is_contiguous() or xcal.dim() != 3 or xcal.shape[2] != K:
        raise ValueError("xcal must be a contiguous CUDA float16 tensor [Bc,T,K]")
    Bc, T = int(xcal.shape[0]), int(xcal.shape[1])
    w_q_packed = _host(w_q_packed, np.uint8)
    N = int(w_q_packed.shape[0])
    if w_q_packed.shape != (N, (K + 1) // 2):
        raise ValueError("packed w_q must be [N, (K+1)//2] bytes")
    w_step = _host(w_step, np.float32, (N,))
    s = np.empty(K, np.float32)
    dx = np.empty(T, np.float32)
    _check(L.ptq_calibrate_w4a4(K, N, T, xcal.data_ptr(), Bc, w_q_packed.ctypes.data, w_step.ctypes.data,
                                s.ctypes.data, dx.ctypes.data, _stream_ptr(stream)))
    return s, dx
