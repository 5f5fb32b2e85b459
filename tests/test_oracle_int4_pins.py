"""Pins of the oracle's 4-bit variant (W4A4 of the latency table; the packing step of Appendix B.1):
hand-evaluated bytes of the packing formula, the round trip over every nibble pair, the relation to
the separately pinned 8-bit quantizer, a numpy float32 evaluation, special values, and the no-clip
invariant of the min-max step."""
import os

import numpy as np

import oracle
from paper_2412_20386_b200 import workloads as wl

F32 = np.float32
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "int4_pack.txt")


def test_pack_matches_the_hand_evaluated_bytes():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 10
    for d0, d1, byte in rows:
        got = oracle.pack_int4(np.array([[int(d0), int(d1)]], np.int8))
        assert got.shape == (1, 1) and int(got[0, 0]) == int(byte, 16), (d0, d1, byte)
        assert oracle.unpack_int4(np.array([[int(byte, 16)]], np.uint8), 2).tolist() == [[int(d0), int(d1)]]


def test_pack_round_trip_all_pairs_and_odd_lengths():
    vals = np.arange(-8, 8, dtype=np.int8)
    pairs = np.array([(a, b) for a in vals for b in vals], np.int8)            # all 256 nibble pairs
    packed = oracle.pack_int4(pairs)
    assert len(set(packed[:, 0].tolist())) == 256                             # a bijection onto the bytes
    assert np.array_equal(oracle.unpack_int4(packed, 2), pairs)
    # independent bit arithmetic
    assert np.array_equal(packed[:, 0], ((pairs[:, 1].astype(np.int32) << 4) | (pairs[:, 0].astype(np.int32) & 15)) & 0xff)
    rng = np.random.default_rng(0)
    for cols in (1, 3, 7, 12, 33):
        d = rng.integers(-8, 8, (5, cols)).astype(np.int8)
        p = oracle.pack_int4(d)
        assert p.shape == (5, (cols + 1) // 2)
        if cols % 2:
            assert np.all(p[:, -1] >> 4 == 0)                                 # an odd row ends with a zero high nibble
        assert np.array_equal(oracle.unpack_int4(p, cols), d)
    # row-major: the second row starts in a fresh byte
    d = np.array([[1, 2, 3], [4, 5, 6]], np.int8)
    assert oracle.pack_int4(d).tolist() == [[0x21, 0x03], [0x54, 0x06]]


def test_quantize4_is_the_clipped_eight_bit_code_and_matches_numpy():
    spec = wl.configs()[0][0]
    x = wl.activations(spec, wl.ROLE_EVAL, B=2).reshape(-1, spec.K)
    wq, dw, _ = wl.weights(spec)
    s, dx8 = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    for scale in (1.0, 127.0 / 7.0, 40.0):
        dx = (dx8 * F32(scale)).astype(F32)
        q4 = oracle.quantize4(x, spec.T, s, dx)
        q8 = oracle.quantize(x, spec.T, s, dx)                                # pinned on its own
        assert np.array_equal(q4, np.clip(q8, -8, 7))
        t = np.arange(x.shape[0]) % spec.T
        v = ((x.astype(F32) / s[None, :]).astype(F32) / dx[t][:, None]).astype(F32)
        assert np.array_equal(q4, np.clip(np.rint(v), -8, 7).astype(np.int8))
    assert q4.min() == -8 and q4.max() == 7                                   # the last scale clips on both sides
    # ties to even, clamp and special values on single elements
    one = lambda val, s_=1.0, d_=1.0: oracle.quantize4_one(int(np.array(val, np.float16).view(np.uint16)), s_, d_)
    assert [one(v) for v in (0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 6.5, 7.5, -7.5, -8.5)] == [0, 2, 2, 0, -2, -2, 6, 7, -8, -8]
    assert [one(v) for v in (7.0, 8.0, 100.0, -8.0, -9.0, -100.0)] == [7, 7, 7, -8, -8, -8]
    assert one(np.nan) == 0 and one(np.inf) == 7 and one(-np.inf) == -8


def test_calibrate4_steps_and_no_clip_invariant():
    spec = wl.configs()[1][0]
    xcal = wl.activations(spec, wl.ROLE_CALIB)
    wq8, dw, _ = wl.weights(spec)
    wq4 = np.clip(wq8 // 16, -8, 7).astype(np.int8)
    s, dx = oracle.calibrate4(xcal, wq4, dw)
    s_ref, dx8 = oracle.calibrate(xcal, wq4, dw)
    assert np.array_equal(s, s_ref)
    u = (xcal.astype(F32) / s[None, None, :]).astype(F32)
    mu = np.maximum(np.abs(u).max(axis=(0, 2)), F32(1e-5))
    assert np.array_equal(dx.view(np.uint32), (mu / F32(7)).astype(F32).view(np.uint32))
    q = oracle.quantize4(xcal.reshape(-1, spec.K), spec.T, s, dx).reshape(xcal.shape)
    amax = np.abs(q.astype(np.int32)).max(axis=(0, 2))
    assert np.all(amax == 7) and q.min() >= -7                                # the range is used fully, never clipped
    # end to end equals the composition with the unpacked weights
    x = wl.activations(spec, wl.ROLE_EVAL, B=2).reshape(-1, spec.K)
    y, q, acc = oracle.linear_forward4(x, spec.T, wq4, dw, s, dx, taps=True)
    assert np.array_equal(acc, q.astype(np.int64) @ wq4.astype(np.int64).T)
    assert np.array_equal(y.view(np.uint16), oracle.dequant(acc, spec.T, dx, dw).view(np.uint16))
