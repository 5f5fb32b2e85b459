"""Pins for the CPU oracle: each checks the oracle against something that does
not route through it (numpy evaluations of the same definition, closed forms,
invariants, brute force), chosen so that a dropped term, a wrong sign or index,
or a transposed operand fails at least one of them.  None of these needs a GPU.
"""
import numpy as np
import pytest

import oracle
from paper_2412_20386_b200 import workloads as wl

F32 = np.float32


def all_half_bits():
    return np.arange(65536, dtype=np.uint32).astype(np.uint16)


# --------------------------------------------------------------------------- #
# binary16 conversions                                                         #
# --------------------------------------------------------------------------- #
def test_half_to_float_all_patterns():
    bits = all_half_bits()
    want = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))  # also signs of zero


def test_double_to_half_roundtrip_and_midpoints():
    bits = all_half_bits()
    vals = bits.view(np.float16)
    finite = np.isfinite(vals)
    # every finite half converts to itself
    for b, v in zip(bits[finite][::7], vals[finite][::7]):
        assert oracle.double_to_half_bits(float(v)) == int(b)
    # midpoints between neighbouring positive halves go to the even neighbour, and a
    # nudge either way goes to the nearer neighbour
    pos = np.sort(vals[finite & (vals >= 0)].astype(np.float64))
    lo, hi = pos[:-1], pos[1:]
    mid = (lo + hi) / 2
    rng = np.random.default_rng(0)
    for i in rng.choice(len(mid), 4000, replace=False):
        lo_b = int(np.float16(lo[i]).view(np.uint16))
        hi_b = int(np.float16(hi[i]).view(np.uint16))
        even = lo_b if lo_b % 2 == 0 else hi_b
        assert oracle.double_to_half_bits(mid[i]) == even
        assert oracle.double_to_half_bits(-mid[i]) == (even | 0x8000)
        assert oracle.double_to_half_bits(np.nextafter(mid[i], 0.0)) == lo_b
        assert oracle.double_to_half_bits(np.nextafter(mid[i], np.inf)) == hi_b
    # overflow boundary: 65520 is the midpoint between 65504 and 2^16
    assert oracle.double_to_half_bits(65504.0) == 0x7bff
    assert oracle.double_to_half_bits(np.nextafter(65520.0, 0.0)) == 0x7bff
    assert oracle.double_to_half_bits(65520.0) == 0x7c00
    assert oracle.double_to_half_bits(-1e9) == 0xfc00
    assert oracle.double_to_half_bits(float("inf")) == 0x7c00
    assert oracle.double_to_half_bits(float("nan")) & 0x7c00 == 0x7c00
    assert oracle.double_to_half_bits(float("nan")) & 0x03ff != 0
    assert oracle.double_to_half_bits(-0.0) == 0x8000


def test_double_to_half_random_against_numpy():
    rng = np.random.default_rng(1)
    v = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.uniform(-9, 5, 20000),
                        rng.uniform(-7e-5, 7e-5, 5000)])
    want = v.astype(np.float16).view(np.uint16)
    got = np.array([oracle.double_to_half_bits(float(z)) for z in v], np.uint16)
    assert np.array_equal(got, want)


# --------------------------------------------------------------------------- #
# Q1 quantizer                                                                 #
# --------------------------------------------------------------------------- #
def numpy_quantize(x_half, s, dx):
    """Independent float32 evaluation of the definition: two IEEE divisions,
    round-half-even, clamp, NaN -> 0."""
    with np.errstate(all="ignore"):
        v = (x_half.astype(F32) / F32(s)) / F32(dx)
        r = np.rint(v)
        r = np.where(np.isnan(r), F32(0), np.clip(r, -128, 127))
    return r.astype(np.int8)


SWEEP_PAIRS = [(1.0, 1.0), (0.37, 0.011), (3.0, 0.1), (1.7320508, 0.0078125),
               (123.456, 1.0e-3), (0.0029, 2.5), (7.0, 1.0 / 3.0), (0.9999999, 0.33333334),
               (5.1e-3, 41.0), (2.0, 0.5)]


@pytest.mark.parametrize("s,dx", SWEEP_PAIRS)
def test_quantizer_all_fp16_inputs_vs_numpy_float32(s, dx):
    bits = all_half_bits()
    x = bits.view(np.float16).reshape(-1, 1)
    got = oracle.quantize(x, 1, np.array([s], F32), np.array([dx], F32)).ravel()
    want = numpy_quantize(x.ravel(), s, dx)
    assert np.array_equal(got, want)
    # NaN -> 0 and infinities saturate
    assert got[0x7e00] == 0 and got[0x7c00] == 127 and got[0xfc00] == -128


def test_quantizer_vs_float64_differs_only_near_ties():
    # In real arithmetic the code is rint(x/(s*dx)); the binary32 definition may differ
    # from it only where the exact quotient sits within a few float32 ulps of a .5 tie.
    bits = all_half_bits()
    xh = bits.view(np.float16)
    fin = np.isfinite(xh)
    x = xh[fin].reshape(-1, 1)
    total_diff = 0
    for s, dx in SWEEP_PAIRS:
        got = oracle.quantize(x, 1, np.array([s], F32), np.array([dx], F32)).ravel().astype(np.int64)
        exact = x.ravel().astype(np.float64) / np.float64(F32(s)) / np.float64(F32(dx))
        want = np.clip(np.rint(exact), -128, 127).astype(np.int64)
        diff = got != want
        total_diff += int(diff.sum())
        if diff.any():
            frac = np.abs(exact[diff] - np.floor(exact[diff]) - 0.5)
            assert np.all(frac <= 4 * np.abs(exact[diff]) * 2.0 ** -23)
            assert np.all(np.abs(got[diff] - want[diff]) == 1)
    assert total_diff < 200


def test_quantizer_keeps_the_two_divisions_separate():
    # (x/s)/dx, x/(s*dx) and x*(1/s)*(1/dx) agree except within an ulp of a rounding tie.  Search for
    # inputs where the binary32 results of these formulations give different codes and require the
    # oracle to side with the two-division definition on every one of them.
    rng = np.random.default_rng(21)
    n = 20000
    xh = (rng.standard_normal(n) * 10.0 ** rng.uniform(-2, 2, n)).astype(np.float16)
    xh = xh[np.isfinite(xh) & (xh != 0)]
    xf = xh.astype(F32)
    s = np.exp(rng.uniform(np.log(1e-2), np.log(1e2), xf.size)).astype(F32)
    k = rng.integers(1, 127, xf.size).astype(F32) + F32(0.5)
    u = (xf / s).astype(F32)
    found = []
    for nudge in (-2, -1, 0, 1, 2):                       # steps chosen so that the quotient lands next to a tie
        dx = (np.abs(u) / k).astype(F32)
        for _ in range(abs(nudge)):
            dx = np.nextafter(dx, F32(np.inf) if nudge > 0 else F32(0)).astype(F32)
        ok = np.isfinite(dx) & (dx > 0)
        two = np.clip(np.rint((xf / s).astype(F32) / dx), -128, 127)
        one = np.clip(np.rint(xf / (s * dx).astype(F32)), -128, 127)
        rec = np.clip(np.rint((xf * (F32(1) / s).astype(F32)).astype(F32) * (F32(1) / dx).astype(F32)), -128, 127)
        for idx in np.nonzero(ok & ((two != one) | (two != rec)))[0][:60]:
            found.append((xh[idx], s[idx], dx[idx], int(two[idx])))
    assert len(found) >= 40, "search found too few discriminating inputs (%d)" % len(found)
    for x, s, dx, want in found:
        got = oracle.quantize_one(int(np.float16(x).view(np.uint16)), float(s), float(dx))
        assert got == want, (float(x), float(s), float(dx), got, want)


def test_quantizer_ties_clamp_and_specials():
    one = np.array([1.0], F32)

    def q(vals, s=1.0, dx=1.0):
        x = np.array(vals, np.float16).reshape(-1, 1)
        return oracle.quantize(x, 1, np.array([s], F32), np.array([dx], F32)).ravel().tolist()

    # ties go to the even integer (power-of-two scales keep the quotients exact)
    assert q([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5]) == [0, 2, 2, 0, -2, -2, 4]
    assert q([1.0, 3.0, 5.0, -3.0], s=0.5, dx=4.0) == [0, 2, 2, -2]   # quotients .5 1.5 2.5 -1.5
    # clamp to [-128, 127]
    assert q([127.0, 127.5, 128.5, 1e4, -127.5, -128.0, -128.5, -1e4]) == [127, 127, 127, 127, -128, -128, -128, -128]
    assert q([np.inf, -np.inf, np.nan]) == [127, -128, 0]
    assert q([0.0, -0.0]) == [0, 0]
    # smallest subnormal half survives two divisions by small scales
    assert q([2.0 ** -24], s=2.0 ** -12, dx=2.0 ** -12) == [1]
    assert one[0] == 1.0


def test_quantizer_monotone_and_odd():
    bits = all_half_bits()
    xh = bits.view(np.float16)
    fin = np.isfinite(xh)
    order = np.argsort(xh[fin].astype(np.float64), kind="stable")
    xs = xh[fin][order].reshape(-1, 1)
    for s, dx in SWEEP_PAIRS[:5]:
        q = oracle.quantize(xs, 1, np.array([s], F32), np.array([dx], F32)).ravel().astype(np.int32)
        assert np.all(np.diff(q) >= 0)
        qn = oracle.quantize(-xs, 1, np.array([s], F32), np.array([dx], F32)).ravel().astype(np.int32)
        sym = (q > -128) & (qn > -128)
        assert np.array_equal(qn[sym], -q[sym])


def test_quantizer_indexes_token_position_and_channel():
    # distinct power-of-two s[k] and dx[t]: the code equals x / (s[k] dx[m mod T]) exactly, so
    # swapping the roles of k and t, or using m instead of m mod T, changes the result.
    T, K, B = 3, 4, 2
    s = np.array([1, 2, 4, 8], F32)
    dx = np.array([1, 0.5, 0.25], F32)
    x = np.full((B * T, K), 16.0, np.float16)
    q = oracle.quantize(x, T, s, dx)
    want = np.array([[16.0 / (s[k] * dx[m % T]) for k in range(K)] for m in range(B * T)])
    assert np.array_equal(q.astype(np.float64), np.clip(want, -128, 127))


# --------------------------------------------------------------------------- #
# G1 integer contraction                                                       #
# --------------------------------------------------------------------------- #
def test_int_matmul_brute_force_tiny():
    rng = np.random.default_rng(2)
    for (M, K, N) in [(1, 1, 1), (2, 3, 4), (5, 8, 3), (8, 7, 8)]:
        q = rng.integers(-128, 128, (M, K)).astype(np.int8)
        w = rng.integers(-127, 128, (N, K)).astype(np.int8)
        acc = oracle.int_matmul(q, w)
        for m in range(M):
            for n in range(N):
                assert int(acc[m, n]) == sum(int(q[m, k]) * int(w[n, k]) for k in range(K))


def test_int_matmul_vs_numpy_int64_and_float64():
    rng = np.random.default_rng(3)
    M, K, N = 257, 1536, 131
    q = rng.integers(-128, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    acc = oracle.int_matmul(q, w)
    assert np.array_equal(acc.astype(np.int64), q.astype(np.int64) @ w.astype(np.int64).T)
    assert np.array_equal(acc.astype(np.float64), q.astype(np.float64) @ w.astype(np.float64).T)


def test_int_matmul_one_hot_and_extremes():
    rng = np.random.default_rng(4)
    K, N = 37, 11
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    q = np.eye(K, dtype=np.int8)                 # row m selects column m of Wq
    assert np.array_equal(oracle.int_matmul(q, w), w.T.astype(np.int32))
    K = 1536
    q = np.full((2, K), 127, np.int8)
    w = np.full((3, K), 127, np.int8)
    assert np.all(oracle.int_matmul(q, w) == K * 16129)
    q[:] = -128
    assert np.all(oracle.int_matmul(q, w) == -K * 128 * 127)


# --------------------------------------------------------------------------- #
# E1 dequantization                                                            #
# --------------------------------------------------------------------------- #
def half_ulp_distance(a, b):
    """Distance in units of binary16 ulps for finite same-sign-or-zero-adjacent values."""
    def key(h):
        u = h.view(np.uint16).astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7fff), u & 0x7fff)
    return np.abs(key(a) - key(b))


def test_dequant_equals_product_of_dequantized_operands():
    # diag(dW) (Wq Xq) diag(dX) == (diag(dW) Wq) (Xq diag(dX))   (Sec. 5.1)
    rng = np.random.default_rng(5)
    M, K, N, T = 90, 96, 40, 9
    q = rng.integers(-128, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    dx = rng.uniform(1e-3, 1e-1, T).astype(F32)
    dw = rng.uniform(1e-3, 1e-2, N).astype(F32)
    bias = rng.standard_normal(N).astype(F32)
    acc = oracle.int_matmul(q, w)
    t = np.arange(M) % T
    xd = q.astype(np.float64) * dx[t].astype(np.float64)[:, None]
    wd = w.astype(np.float64) * dw.astype(np.float64)[:, None]
    for b in (None, bias):
        y = oracle.dequant(acc, T, dx, dw, b)
        ref = xd @ wd.T + (0 if b is None else b.astype(np.float64)[None, :])
        ref16 = ref.astype(np.float16)
        d = half_ulp_distance(y, ref16)
        assert d.max() <= 1
        assert (d == 0).mean() > 0.995


def test_dequant_power_of_two_steps_exact():
    rng = np.random.default_rng(6)
    M, N, T = 33, 17, 5
    acc = rng.integers(-2000, 2000, (M, N)).astype(np.int32)
    dx = (2.0 ** rng.integers(-6, 0, T)).astype(F32)
    dw = (2.0 ** rng.integers(-6, 0, N)).astype(F32)
    y = oracle.dequant(acc, T, dx, dw)
    t = np.arange(M) % T
    ref = (acc.astype(np.float64) * dx[t][:, None] * dw[None, :]).astype(np.float16)
    assert np.array_equal(y.view(np.uint16), ref.view(np.uint16))
    # overflow goes to infinity, not to the largest finite half
    big = np.array([[2 ** 24]], np.int32)
    assert np.isposinf(oracle.dequant(big, 1, np.array([1.0], F32), np.array([1.0], F32))[0, 0])
    assert np.isneginf(oracle.dequant(-big, 1, np.array([1.0], F32), np.array([1.0], F32))[0, 0])


# --------------------------------------------------------------------------- #
# Whole path                                                                   #
# --------------------------------------------------------------------------- #
def test_closed_form_integer_inputs_reproduce_exact_integer_matmul():
    # s = 1, dx = 1, dw = 1, integer-valued activations: q == x and y == fp16(sum x Wq)
    rng = np.random.default_rng(7)
    B, T, K, N = 3, 5, 24, 10
    xi = rng.integers(-128, 128, (B * T, K))
    wq = rng.integers(-3, 4, (N, K)).astype(np.int8)
    x = xi.astype(np.float16)
    ones = lambda n: np.ones(n, F32)
    y, q, acc = oracle.linear_forward(x, T, wq, ones(N), ones(K), ones(T), taps=True)
    assert np.array_equal(q.astype(np.int64), xi)
    exact = xi @ wq.astype(np.int64).T
    assert np.array_equal(acc.astype(np.int64), exact)
    assert np.array_equal(y.view(np.uint16), exact.astype(np.float64).astype(np.float16).view(np.uint16))


def test_forward_rows_equals_composition_and_row_ranges():
    spec = wl.configs()[0][0]
    x = wl.activations(spec, wl.ROLE_EVAL, B=2).reshape(-1, spec.K)
    wq, dw, _ = wl.weights(spec)
    s, dx = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    bias = np.linspace(-1, 1, spec.N).astype(F32)
    q = oracle.quantize(x, spec.T, s, dx)
    acc = oracle.int_matmul(q, wq)
    y = oracle.dequant(acc, spec.T, dx, dw, bias)
    y2, q2, acc2 = oracle.linear_forward(x, spec.T, wq, dw, s, dx, bias, taps=True)
    assert np.array_equal(q, q2) and np.array_equal(acc, acc2)
    assert np.array_equal(y.view(np.uint16), y2.view(np.uint16))
    y3 = oracle.linear_forward(x, spec.T, wq, dw, s, dx, bias, rows=(190, 230))
    assert np.array_equal(y3.view(np.uint16), y[190:230].view(np.uint16))


def test_smoothing_invariance_and_quantization_error_bound():
    # Eq. smooth: (W diag(s)) (diag(s)^-1 X) = W X.  With the folded weight quantized per output
    # channel (Sec. 2.3) the oracle's output must stay within the worst-case rounding bound of
    # the float64 product x W^T; a wrong index, sign or transposition breaks the bound.
    rng = np.random.default_rng(8)
    B, T, K, N = 4, 7, 48, 20
    M = B * T
    x = (rng.standard_t(3, (M, K)) * np.exp(rng.normal(0, 0.5, (M, 1)))).astype(np.float16)
    W = rng.standard_normal((N, K)) * 0.05
    s = np.sqrt(np.abs(x.astype(np.float64)).max(0) / np.abs(W).max(0)).astype(F32)
    s64 = s.astype(np.float64)
    x64 = x.astype(np.float64)
    Wf = W * s64[None, :]
    assert np.allclose((x64 / s64) @ Wf.T, x64 @ W.T, rtol=1e-12, atol=1e-12)
    dw = (np.abs(Wf).max(1) / 127).astype(F32)
    wq = np.clip(np.rint(Wf / dw.astype(np.float64)[:, None]), -127, 127).astype(np.int8)
    t = np.arange(M) % T
    u = x64 / s64
    dx = np.array([np.abs(u[t == i]).max() / 127 for i in range(T)]).astype(F32)
    y, q, _ = oracle.linear_forward(x, T, wq, dw, s, dx, taps=True)
    assert np.abs(q.astype(np.int32)).max() <= 127 + 1
    dxm = dx.astype(np.float64)[t][:, None]
    # reconstruction: dequantized code times s is within half a step of x
    assert np.all(np.abs(q * dxm * s64 - x64) <= 0.5 * dxm * s64 * (1 + 1e-6) + 1e-12)
    eu = 0.5 * dxm * (1 + 1e-6) * np.ones_like(u)
    ew = 0.5 * dw.astype(np.float64)[:, None] * (1 + 1e-6) * np.ones_like(Wf)
    bound = eu @ np.abs(Wf).T + np.abs(u) @ ew.T + eu @ ew.T
    ref = x64 @ W.T
    err = np.abs(y.astype(np.float64) - ref)
    assert np.all(err <= bound + np.abs(ref) * 2.0 ** -10 + 1e-6)
    # and the bound is not vacuous: the quantized output tracks the float product closely
    assert np.linalg.norm(y.astype(np.float64) - ref) / np.linalg.norm(ref) < 0.02


# --------------------------------------------------------------------------- #
# Q0 calibration                                                               #
# --------------------------------------------------------------------------- #
def numpy_calibrate(xcal, wq, dw):
    Bc, T, K = xcal.shape
    xf = xcal.astype(F32)
    floor_ = F32(1e-5)
    max_x = np.maximum(np.abs(xf).max(axis=(0, 1)), floor_)
    max_w = np.maximum((np.abs(wq.astype(F32)) * dw[:, None].astype(F32)).max(axis=0), floor_)
    s = np.sqrt((max_x / max_w).astype(F32)).astype(F32)
    u = (xf / s[None, None, :]).astype(F32)
    mu = np.maximum(np.abs(u).max(axis=(0, 2)), floor_)
    return s, (mu / F32(127)).astype(F32)


def test_calibrate_vs_numpy_float32_and_no_clip_invariant():
    spec = wl.configs()[1][1]          # x_proj 384 -> 44
    xcal = wl.activations(spec, wl.ROLE_CALIB)
    wq, dw, _ = wl.weights(spec)
    s, dx = oracle.calibrate(xcal, wq, dw)
    s_np, dx_np = numpy_calibrate(xcal, wq, dw)
    assert np.array_equal(s.view(np.uint32), s_np.view(np.uint32))
    assert np.array_equal(dx.view(np.uint32), dx_np.view(np.uint32))
    # the calibration batch itself never clips, and every token position reaches +-127
    q = oracle.quantize(xcal.reshape(-1, spec.K), spec.T, s, dx).astype(np.int32)
    assert q.min() >= -127 and q.max() <= 127
    per_t = np.abs(q).reshape(-1, spec.T, spec.K).max(axis=(0, 2))
    assert np.all(per_t == 127)


def test_calibrate_degenerate_channels_and_positions():
    T, K, N = 3, 4, 2
    xcal = np.zeros((2, T, K), np.float16)
    xcal[:, 1, 2] = 3.0                                   # only one live channel / position
    wq = np.array([[10, 0, -20, 0], [5, 0, 40, 0]], np.int8)
    dw = np.array([0.01, 0.02], F32)
    s, dx = oracle.calibrate(xcal, wq, dw)
    assert np.all(np.isfinite(s)) and np.all(s > 0) and np.all(dx > 0)
    s_np, dx_np = numpy_calibrate(xcal, wq, dw)
    assert np.array_equal(s, s_np) and np.array_equal(dx, dx_np)
    # channel 2: maxX = 3, maxW = max(20*.01, 40*.02) = 0.8
    assert s[2] == F32(np.sqrt(F32(3.0) / F32(0.8)))
    # dead channel with dead weights: sqrt(1e-5/1e-5) = 1
    assert s[1] == F32(1.0)
    assert dx[0] == F32(F32(1e-5) / F32(127))


def test_calibrate_per_tensor_vs_numpy_float32_and_invariants():
    # the per-tensor static comparator: one step for the whole tensor (latency table of Sec. 6, Fig. 5)
    spec = wl.configs()[1][1]          # x_proj 384 -> 44
    xcal = wl.activations(spec, wl.ROLE_CALIB)
    wq, dw, _ = wl.weights(spec)
    s, delta = oracle.calibrate_per_tensor(xcal, wq, dw)
    s_np, dx_np = numpy_calibrate(xcal, wq, dw)
    assert np.array_equal(s.view(np.uint32), s_np.view(np.uint32))
    # independent numpy float32 evaluation of max|x/s| / 127 over the whole batch
    u = (xcal.astype(F32) / s_np[None, None, :]).astype(F32)
    want = F32(max(F32(np.abs(u).max()), F32(1e-5)) / F32(127))
    assert F32(delta).view(np.uint32) == want.view(np.uint32)
    # it is the largest of the per-position steps (division by 127 is monotonic), strictly above most of them
    assert delta == dx_np.max() and (dx_np < delta).sum() >= spec.T - 2
    # one step for all positions never clips the calibration batch, reaches +-127 somewhere, and wastes
    # range at the quiet positions: that is what the per-token steps repair (Sec. 4.1 and 5.1)
    q = oracle.quantize(xcal.reshape(-1, spec.K), spec.T, s, np.full(spec.T, delta, F32)).astype(np.int32)
    assert q.min() >= -127 and q.max() <= 127 and np.abs(q).max() == 127
    per_t = np.abs(q).reshape(-1, spec.T, spec.K).max(axis=(0, 2))
    assert (per_t < 127).sum() >= spec.T - 2 and per_t[98] < 32          # the class-token row uses a fraction of the range
    # degenerate batch: the floor
    z = np.zeros((2, 3, 4), np.float16)
    _, d0 = oracle.calibrate_per_tensor(z, np.ones((2, 4), np.int8), np.array([0.01, 0.02], F32))
    assert d0 == F32(F32(1e-5) / F32(127))


# --------------------------------------------------------------------------- #
# input generator                                                              #
# --------------------------------------------------------------------------- #
def test_workloads_are_deterministic_and_shaped():
    cfg = wl.configs()
    assert [len(cfg[i]) for i in range(5)] == [1, 96, 2, 2, 8]
    spec = cfg[1][2]
    assert (spec.K, spec.N, spec.bias, spec.T, spec.B) == (12, 384, True, 197, 64)
    a = wl.activations(spec, wl.ROLE_EVAL, B=2)
    b = wl.activations(spec, wl.ROLE_EVAL, B=3)
    assert a.dtype == np.float16 and a.shape == (2, 197, 12)
    assert np.array_equal(a, b[:2])                         # prefix-stable in the batch
    assert not np.array_equal(a, wl.activations(spec, wl.ROLE_CALIB, B=2))
    wq, dw, bias = wl.weights(spec)
    assert wq.dtype == np.int8 and wq.min() >= -127 and wq.max() <= 127
    assert dw.dtype == F32 and dw.min() >= 1e-3 and dw.max() <= 1e-2 and bias.shape == (384,)
    assert np.all(np.isfinite(a.astype(np.float32)))
    # class-token position is an order of magnitude quieter than its neighbours on average
    big = wl.activations(cfg[0][0], wl.ROLE_EVAL, B=4).astype(np.float64)
    g, o = wl.structure(cfg[0][0])
    assert g[98] < 0.5 * np.median(g) and (o > 1).sum() == 4
    assert np.abs(big[:, 98]).mean() < np.abs(big).mean()


# --------------------------------------------------------------------------- #
# comparator: per-token dynamic quantization                                   #
# --------------------------------------------------------------------------- #
def test_dynamic_quantizer_vs_numpy_and_invariants():
    spec = wl.configs()[0][0]
    x = wl.activations(spec, wl.ROLE_EVAL, B=3).reshape(-1, spec.K)
    x[5] = 0                                                    # a dead row: floored step, all-zero codes
    wq, dw, _ = wl.weights(spec)
    s, _ = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    q, dx_row = oracle.quantize_dynamic(x, s)
    u = (x.astype(F32) / s[None, :]).astype(F32)
    mu = np.maximum(np.abs(u).max(axis=1), F32(1e-5))
    dx_np = (mu / F32(127)).astype(F32)
    assert np.array_equal(dx_row.view(np.uint32), dx_np.view(np.uint32))
    q_np = np.clip(np.rint((u / dx_np[:, None]).astype(F32)), -128, 127).astype(np.int8)
    assert np.array_equal(q, q_np)
    # every live row uses the full range and never needs the clamp
    live = np.abs(x.astype(np.float32)).max(axis=1) > 0
    assert np.all(np.abs(q[live].astype(np.int32)).max(axis=1) == 127) and q.min() >= -127
    assert np.all(q[5] == 0) and dx_row[5] == F32(F32(1e-5) / F32(127))
    # the static quantizer fed with the row steps (T = M) gives the same codes
    assert np.array_equal(oracle.quantize(x, x.shape[0], s, dx_row), q)
    # scaling a row by a power of two scales its step and leaves its codes alone
    x2 = x.copy()
    x2[7] = (x[7].astype(np.float32) * 4).astype(np.float16)
    q2, dx2 = oracle.quantize_dynamic(x2, s)
    assert np.array_equal(q2[7], q[7]) and dx2[7] == F32(4) * dx_row[7]
    # end to end equals the composition with T = M
    y, qq, acc, dd = oracle.linear_forward_dynamic(x, wq, dw, s, taps=True)
    assert np.array_equal(acc, oracle.int_matmul(q, wq))
    assert np.array_equal(y.view(np.uint16), oracle.dequant(acc, x.shape[0], dx_row, dw).view(np.uint16))
