"""Pins for the oracle's asymmetric PTS functions (step and zero offset per token position, Sec. 5.1
with the quantizer form of Sec. 2.3), independent of the oracle's own code."""
import numpy as np
import pytest

import oracle
from paper_2412_20386_b200 import workloads as wl

F32 = np.float32


def numpy_quantize_asym(x_half, s, dx, z):
    with np.errstate(all="ignore"):
        v = (x_half.astype(F32) / F32(s)) / F32(dx)
        r = np.rint(v).astype(np.float64) + z
        r = np.where(np.isnan(r), float(z), np.clip(r, 0, 255))
    return r.astype(np.uint8)


@pytest.mark.parametrize("s,dx,z", [(1.0, 1.0, 0), (0.37, 0.011, 128), (3.0, 0.1, 17), (1.7320508, 0.0078125, 255),
                                    (0.0029, 2.5, 100), (7.0, 1.0 / 3.0, 200)])
def test_asym_quantizer_all_fp16_inputs_vs_numpy_float32(s, dx, z):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    x = bits.view(np.float16).reshape(-1, 1)
    got = oracle.quantize_asym(x, 1, np.array([s], F32), np.array([dx], F32), np.array([z], np.int32)).ravel()
    assert np.array_equal(got, numpy_quantize_asym(x.ravel(), s, dx, z))
    assert got[0x7e00] == z and got[0x7c00] == 255 and got[0xfc00] == 0        # NaN, +inf, -inf


def test_asym_with_offset_128_reproduces_symmetric_codes_and_accumulators():
    spec = wl.configs()[0][0]
    x = wl.activations(spec, wl.ROLE_EVAL, B=2).reshape(-1, spec.K)
    wq, dw, _ = wl.weights(spec)
    s, dx = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    z = np.full(spec.T, 128, np.int32)
    q = oracle.quantize(x, spec.T, s, dx).astype(np.int32)
    c = oracle.quantize_asym(x, spec.T, s, dx, z).astype(np.int32)
    assert np.array_equal(c - 128, q)                      # [-128,127] + 128 = [0,255]: same clipping
    assert np.array_equal(oracle.int_matmul_asym(c.astype(np.uint8), z, spec.T, wq),
                          oracle.int_matmul(q.astype(np.int8), wq))


def test_asym_indices_ties_and_clamp():
    T, K = 3, 4
    s = np.array([1, 2, 4, 8], F32)
    dx = np.array([1, 0.5, 0.25], F32)
    z = np.array([10, 20, 30], np.int32)
    x = np.full((2 * T, K), 16.0, np.float16)
    c = oracle.quantize_asym(x, T, s, dx, z)
    want = np.array([[16.0 / (s[k] * dx[m % T]) + z[m % T] for k in range(K)] for m in range(2 * T)])
    assert np.array_equal(c.astype(np.float64), np.clip(want, 0, 255))
    one = np.ones(1, F32)
    q = lambda vals, zz: oracle.quantize_asym(np.array(vals, np.float16).reshape(-1, 1), 1, one, one,
                                              np.array([zz], np.int32)).ravel().tolist()
    assert q([0.5, 1.5, 2.5, -0.5, -1.5], 5) == [5, 7, 7, 5, 3]           # ties to even BEFORE the offset
    assert q([250.0, 251.0, -5.0, -6.0, 1e4, -1e4], 5) == [255, 255, 0, 0, 255, 0]
    # the offset is added to the ROUNDED integer: 0.5 / 0.99999994 is just above the tie, which a
    # binary32 addition of 128 before rounding would erase
    just_below_one = np.array([np.nextafter(F32(1), F32(0))], F32)
    qq = lambda vals, zz: oracle.quantize_asym(np.array(vals, np.float16).reshape(-1, 1), 1, one, just_below_one,
                                               np.array([zz], np.int32)).ravel().tolist()
    assert qq([0.5, -0.5], 128) == [129, 127]


def test_asym_matmul_brute_force_and_closed_form():
    rng = np.random.default_rng(31)
    M, K, N, T = 7, 9, 5, 3
    c = rng.integers(0, 256, (M, K)).astype(np.uint8)
    z = rng.integers(0, 256, T).astype(np.int32)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    acc = oracle.int_matmul_asym(c, z, T, w)
    for m in range(M):
        for n in range(N):
            assert int(acc[m, n]) == sum((int(c[m, k]) - int(z[m % T])) * int(w[n, k]) for k in range(K))
    # closed form: s = dx = dw = 1, integer activations inside the offset range: exact integer matmul
    xi = rng.integers(-10, 246, (2 * T, K))
    zz = np.full(T, 10, np.int32)
    ones = lambda n: np.ones(n, F32)
    y, cc, acc = oracle.linear_forward_asym(xi.astype(np.float16), T, w, ones(N), ones(K), ones(T), zz, taps=True)
    assert np.array_equal(cc.astype(np.int64), xi + 10)
    exact = xi @ w.astype(np.int64).T
    assert np.array_equal(acc.astype(np.int64), exact)
    assert np.array_equal(y.view(np.uint16), exact.astype(np.float64).astype(np.float16).view(np.uint16))


def numpy_calibrate_asym(xcal, wq, dw):
    Bc, T, K = xcal.shape
    xf = xcal.astype(F32)
    floor_ = F32(1e-5)
    max_x = np.maximum(np.abs(xf).max(axis=(0, 1)), floor_)
    max_w = np.maximum((np.abs(wq.astype(F32)) * dw[:, None].astype(F32)).max(axis=0), floor_)
    s = np.sqrt((max_x / max_w).astype(F32)).astype(F32)
    u = (xf / s[None, None, :]).astype(F32)
    lo = np.minimum(u.min(axis=(0, 2)), F32(0))
    hi = np.maximum(u.max(axis=(0, 2)), F32(0))
    dx = (np.maximum((hi - lo).astype(F32), floor_) / F32(255)).astype(F32)
    z = np.clip(np.rint((-lo / dx).astype(F32)), 0, 255).astype(np.int32)
    return s, dx, z


def test_asym_calibration_vs_numpy_and_never_clips():
    spec = wl.configs()[1][3]
    xcal = wl.activations(spec, wl.ROLE_CALIB) + np.float16(0.75)          # skewed range: offset away from 128
    wq, dw, _ = wl.weights(spec)
    s, dx, z = oracle.calibrate_asym(xcal, wq, dw)
    s_np, dx_np, z_np = numpy_calibrate_asym(xcal, wq, dw)
    assert np.array_equal(s.view(np.uint32), s_np.view(np.uint32))
    assert np.array_equal(dx.view(np.uint32), dx_np.view(np.uint32))
    assert np.array_equal(z, z_np) and z.min() >= 0 and z.max() <= 255
    c = oracle.quantize_asym(xcal.reshape(-1, spec.K), spec.T, s, dx, z).astype(np.int32).reshape(-1, spec.T, spec.K)
    # the calibration batch spans (almost) the whole code range at every position and never needs clipping:
    # the unclipped integer round(v) + z already lies in [0, 255] up to one step of rounding at each end
    v = (xcal.astype(F32) / s[None, None, :]) / dx[None, :, None]
    raw = np.rint(v).astype(np.int64) + z[None, :, None]
    assert raw.min() >= -1 and raw.max() <= 256
    assert np.all(c.min(axis=(0, 2)) <= 1) and np.all(c.max(axis=(0, 2)) >= 254)
    # reconstruction: (c - z) dx s is within half a step of x wherever nothing clipped
    rec = (c - z[None, :, None]) * dx[None, :, None].astype(np.float64) * s[None, None, :].astype(np.float64)
    ok = (raw >= 0) & (raw <= 255)
    err = np.abs(rec - xcal.astype(np.float64))
    bound = 0.5 * dx[None, :, None].astype(np.float64) * s[None, None, :] * (1 + 1e-5) + 1e-9
    assert np.all(err[ok] <= np.broadcast_to(bound, err.shape)[ok])


def test_asym_calibration_range_contains_zero_and_degenerate_positions():
    T, K = 3, 4
    xcal = np.zeros((2, T, K), np.float16)
    xcal[:, 0, :] = [[2, 3, 4, 5], [2.5, 3.5, 4.5, 5]]       # all positive: lo is pinned to 0, offset 0
    xcal[:, 1, :] = [[-2, -3, -4, -5], [-2.5, -3.5, -4.5, -5]]  # all negative: hi is pinned to 0, offset 255
    wq = np.array([[10, 10, 10, 10]], np.int8)
    dw = np.array([0.1], F32)                                  # maxW = 1 -> s = sqrt(5)
    s, dx, z = oracle.calibrate_asym(xcal, wq, dw)
    s_np, dx_np, z_np = numpy_calibrate_asym(xcal, wq, dw)
    assert np.array_equal(s, s_np) and np.array_equal(dx, dx_np) and np.array_equal(z, z_np)
    assert z.tolist() == [0, 255, 0]
    hi = F32(5) / s[3]
    assert dx[0] == F32(hi / F32(255)) and dx[1] == dx[0]
    assert dx[2] == F32(F32(1e-5) / F32(255))                  # dead position: floored range


def test_asym_forward_rows_equals_composition():
    spec = wl.configs()[0][0]
    x = wl.activations(spec, wl.ROLE_EVAL, B=2).reshape(-1, spec.K)
    wq, dw, _ = wl.weights(spec)
    s, dx, z = oracle.calibrate_asym(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    bias = np.linspace(-1, 1, spec.N).astype(F32)
    c = oracle.quantize_asym(x, spec.T, s, dx, z)
    acc = oracle.int_matmul_asym(c, z, spec.T, wq)
    y = oracle.dequant(acc, spec.T, dx, dw, bias)
    y2, c2, acc2 = oracle.linear_forward_asym(x, spec.T, wq, dw, s, dx, z, bias, taps=True)
    assert np.array_equal(c, c2) and np.array_equal(acc, acc2) and np.array_equal(y.view(np.uint16), y2.view(np.uint16))
    y3 = oracle.linear_forward_asym(x, spec.T, wq, dw, s, dx, z, bias, rows=(100, 260))
    assert np.array_equal(y3.view(np.uint16), y[100:260].view(np.uint16))
