"""Pins of the oracle's step-size search (Sec. 5.2, second stage: grid search of the activation step
that minimises the L2 distance between the smoothed activations and their dequantized codes, per token
position).  None of them re-types the oracle's loop: exact rational arithmetic on tiny inputs, closed
forms (zero loss on grid points, the Delta^2/12 law), planted ties, an outlier that makes truncation
win, and the link to the separately pinned quantizer."""
from fractions import Fraction

import numpy as np

import oracle

F32 = np.float32


def rn32(fr: Fraction) -> Fraction:
    """Round an exact rational to the nearest binary32 (ties to even), without double rounding."""
    if fr == 0:
        return Fraction(0)
    c = F32(float(fr))
    cands = {c, np.nextafter(c, F32(np.inf)), np.nextafter(c, F32(-np.inf))}
    best = None
    for v in cands:
        d = abs(Fraction(float(v)) - fr)
        even = (int(np.array(v, F32).view(np.uint32)) & 1) == 0
        key = (d, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, Fraction(float(v)))
    return best[1]


def exact_losses(x, s, base, n_grid, j_lo):
    """loss[t][j] as exact rationals, with binary32 roundings where the definition has them."""
    Bc, T, K = x.shape
    out = []
    for t in range(T):
        row = []
        for j in range(j_lo, n_grid + 1):
            ratio = F32(F32(j) / F32(n_grid))
            delta = F32(base[t] * ratio)
            acc = Fraction(0)
            for b in range(Bc):
                for k in range(K):
                    u = F32(F32(x[b, t, k]) / s[k])
                    if not np.isfinite(u):
                        continue
                    v = F32(u / delta)
                    q = int(min(max(np.rint(v), -128), 127))
                    e = rn32(Fraction(float(u)) - Fraction(float(delta)) * q)
                    acc += e * e
            row.append(acc)
        out.append(row)
    return out


def test_search_matches_exact_rational_brute_force():
    rng = np.random.default_rng(3)
    Bc, T, K = 2, 3, 8
    x = (rng.standard_normal((Bc, T, K)) * np.array([1.0, 4.0, 0.25])[None, :, None]).astype(np.float16)
    x[0, 1, 2] = 40.0                                   # an outlier: clipping matters for small ratios
    s = np.exp(rng.uniform(-1, 1, K)).astype(F32)
    base = (np.abs(x.astype(F32) / s[None, None, :]).max(axis=(0, 2)) / F32(127)).astype(F32)
    n_grid, j_lo = 10, 2
    dx, best, loss = oracle.search_act_step(x, s, base, n_grid, j_lo)
    ref = exact_losses(x, s, base, n_grid, j_lo)
    for t in range(T):
        for c in range(n_grid - j_lo + 1):
            r = float(ref[t][c])
            assert abs(loss[t, c] - r) <= 1e-12 * max(r, 1e-30), (t, c)
        least = min(ref[t])
        j_ref = max(j for j in range(j_lo, n_grid + 1) if ref[t][j - j_lo] == least)
        assert best[t] == j_ref
        assert dx[t] == F32(base[t] * F32(F32(j_ref) / F32(n_grid)))


def test_search_zero_loss_on_grid_points_and_ties_keep_the_largest_ratio():
    # activations that are integer multiples of the full step: no error at ratio 1, and none at
    # ratios 1/2 and 1/4 either as long as nothing clips -> a three-way tie, the largest j wins
    T, K = 2, 32
    base = np.array([2.0 ** -3, 2.0 ** -5], F32)
    m = np.arange(-15, 17).astype(np.float64)              # |4 m| <= 64 < 127: no clipping even at ratio 1/4
    x = np.stack([m * base[0], m * base[1]])[None].astype(np.float16)
    dx, best, loss = oracle.search_act_step(x, np.ones(K, F32), base, 4, 1)
    assert np.all(loss[:, [0, 1, 3]] == 0.0)               # j = 1, 2, 4
    assert np.all(loss[:, 2] > 0.0)                        # j = 3: step 3/4 base does not divide the data
    assert best.tolist() == [4, 4] and np.array_equal(dx, base)
    # with |m| up to 60 the ratio 1/4 clips (4 * 60 > 127) and 1/2 does not: still j = 4, loss[j=1] > 0
    m2 = np.linspace(-60, 60, K).round()
    x2 = np.stack([m2 * base[0], m2 * base[1]])[None].astype(np.float16)
    _, best2, loss2 = oracle.search_act_step(x2, np.ones(K, F32), base, 4, 1)
    assert np.all(loss2[:, 0] > 0) and np.all(loss2[:, 1] == 0) and np.all(loss2[:, 3] == 0)
    assert best2.tolist() == [4, 4]
    # all-zero activations: every candidate has zero loss
    _, best0, loss0 = oracle.search_act_step(np.zeros((2, 3, 8), np.float16), np.ones(8, F32),
                                             np.full(3, 1e-5 / 127, F32), 100, 20)
    assert np.all(loss0 == 0) and np.all(best0 == 100)


def test_search_loss_follows_the_uniform_rounding_error_law():
    # without clipping, rounding errors are uniform in [-Delta/2, Delta/2]: mean e^2 = Delta^2 / 12
    rng = np.random.default_rng(11)
    Bc, T, K = 16, 3, 2048
    x = rng.uniform(-1, 1, (Bc, T, K)).astype(np.float16)
    base = np.full(T, 4.0 / 127, F32)                      # range +-4: nothing clips for j >= 25 of 100
    _, _, loss = oracle.search_act_step(x, np.ones(K, F32), base, 100, 25)
    j = np.arange(25, 101)
    delta = (4.0 / 127) * j / 100.0
    expect = Bc * K * delta ** 2 / 12.0
    assert np.all(np.abs(loss / expect[None, :] - 1.0) < 0.03)
    # and the smallest step therefore wins
    assert np.all(np.argmin(loss, axis=1) == 0)


def test_search_truncates_when_an_outlier_stretches_the_range():
    rng = np.random.default_rng(17)
    Bc, T, K = 8, 2, 4096
    x = rng.standard_normal((Bc, T, K))
    x[0, 0, 5] = 100.0                                     # one outlier per position,
    x[0, 1, 5] = -100.0                                    # positive in one, negative in the other
    x = x.astype(np.float16)
    s = np.ones(K, F32)
    base = np.full(T, 100.0 / 127, F32)
    dx, best, loss = oracle.search_act_step(x, s, base, 100, 5)
    # independent float64 evaluation of the same objective
    u = x.astype(np.float64)
    ref = np.empty((T, 96))
    for c, jj in enumerate(range(5, 101)):
        d = float(F32(base[0] * F32(F32(jj) / F32(100))))
        q = np.clip(np.rint(u / d), -128, 127)
        ref[:, c] = ((u - d * q) ** 2).sum(axis=(0, 2))
    assert np.allclose(loss, ref, rtol=1e-5)
    assert np.array_equal(best, 5 + np.argmin(ref, axis=1))
    # closed form: clipping the outlier costs 100^2 (1-r)^2, rounding the other n values costs
    # n (r 100/127)^2 / 12; the sum is least at r* = 1 / (1 + n / (12 * 127^2))
    r_star = 1.0 / (1.0 + Bc * K / (12.0 * 127.0 ** 2))
    assert r_star < 0.9 and np.all(np.abs(best / 100.0 - r_star) < 0.03)
    assert np.all(loss[np.arange(T), best - 5] < loss[:, -1])
    assert np.array_equal(dx, (base * (best.astype(F32) / F32(100))).astype(F32))


def test_search_skips_non_finite_values_and_uses_the_pinned_quantizer():
    rng = np.random.default_rng(23)
    Bc, T, K = 4, 5, 64
    x = rng.standard_normal((Bc, T, K)).astype(np.float16)
    x[:, :, :4] = 0                                         # exact zeros: no error at any step
    s = np.exp(rng.uniform(-1, 1, K)).astype(F32)
    base = (np.abs(x.astype(F32) / s).max(axis=(0, 2)) / F32(127)).astype(F32)
    dx, best, loss = oracle.search_act_step(x, s, base, 50, 10)
    x2 = x.copy()
    x2[0, :, 0] = np.inf
    x2[1, :, 1] = -np.inf
    x2[2, :, 2] = np.nan
    dx2, best2, loss2 = oracle.search_act_step(x2, s, base, 50, 10)
    assert np.array_equal(loss, loss2) and np.array_equal(best, best2) and np.array_equal(dx, dx2)
    # the codes inside the loss are those of the quantizer (pinned on its own)
    for jj in (10, 33, 50):
        d = (base * F32(F32(jj) / F32(50))).astype(F32)
        q = oracle.quantize(x.reshape(-1, K), T, s, d).reshape(Bc, T, K).astype(np.float64)
        u = (x.astype(F32) / s).astype(np.float64)
        ref = ((u - d.astype(np.float64)[None, :, None] * q) ** 2).sum(axis=(0, 2))
        assert np.allclose(loss[:, jj - 10], ref, rtol=1e-6)
