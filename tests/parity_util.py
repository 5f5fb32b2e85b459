"""Shared helpers of the GPU parity tests: run one layer through the C ABI and compare it with the
CPU oracle on the same seeded inputs."""
import numpy as np

import oracle
from paper_2412_20386_b200 import workloads as wl

REL_TOL = 2.0 ** -10      # max relative error of the fp16 outputs
ABS_TOL = 1e-3            # near zero


def assert_y_close(y_gpu, y_ref, what=""):
    """Equal if both are the same infinity; otherwise |a-b| <= max(2^-10 |b|, 1e-3)."""
    a = np.asarray(y_gpu).astype(np.float64).ravel()
    b = np.asarray(y_ref).astype(np.float64).ravel()
    assert a.shape == b.shape
    inf = np.isinf(b)
    assert np.array_equal(a[inf], b[inf]), "%s: infinities differ" % what
    d = np.abs(a[~inf] - b[~inf])
    lim = np.maximum(REL_TOL * np.abs(b[~inf]), ABS_TOL)
    bad = d > lim
    assert not bad.any(), "%s: %d of %d outputs out of tolerance (worst %g at ref %g)" % (
        what, int(bad.sum()), d.size, float(d[bad].max()), float(b[~inf][bad][np.argmax(d[bad])]))


def sample_row_blocks(M, rng, n_blocks=6, block=96):
    """Contiguous row ranges covering the first tile, the ragged tail and random interior tiles."""
    if M <= 4 * block:
        return [(0, M)]
    blocks = [(0, block), (M - block, M), (M // 2 - 7, M // 2 - 7 + block)]
    for _ in range(n_blocks - 3):
        m0 = int(rng.integers(0, M - block))
        blocks.append((m0, m0 + block))
    return blocks


def layer_inputs(spec, B=None):
    x = wl.activations(spec, wl.ROLE_EVAL, B=B)
    wq, dw, bias = wl.weights(spec)
    s, dx = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    return x, wq, dw, bias, s, dx


def check_layer(ptq, torch, spec, B=None, flags_list=(0, 1, 2), full=None, seed=0):
    """Forward with taps through the C ABI, once per entry of flags_list (0 = quantize kernel then
    GEMM kernel, 1 = PTQ_FLAG_FUSED_PROLOGUE, 2 = PTQ_FLAG_CTA_PAIR); compare codes and accumulators bit for bit and the fp16
    output within tolerance, on every row (small layers) or on sampled row blocks (large ones)."""
    x, wq, dw, bias, s, dx = layer_inputs(spec, B)
    Bn = x.shape[0]
    M = Bn * spec.T
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xd = torch.from_numpy(x).cuda()
    x2 = x.reshape(M, spec.K)
    if full is None:
        full = M * spec.K * spec.N <= 4e9
    blocks = [(0, M)] if full else sample_row_blocks(M, np.random.default_rng(seed))
    refs = [oracle.linear_forward(x2, spec.T, wq, dw, s, dx, bias, rows=blk, taps=True) for blk in blocks]
    q_all = None if full else oracle.quantize(x2, spec.T, s, dx)
    clip = 0
    for flags in flags_list:
        what = "%s flags=%d" % (spec.name, flags)
        y, q, acc = layer.forward_debug(xd, flags=flags)
        y2 = layer.forward(xd, flags=flags)                   # the production entry point
        torch.cuda.synchronize()
        layer.device_status()
        assert torch.equal(y, y2), "%s: forward and forward_debug disagree" % what
        y = y.cpu().numpy().reshape(M, spec.N)
        q = q.cpu().numpy().reshape(M, spec.K)
        acc = acc.cpu().numpy().reshape(M, spec.N)
        for (m0, m1), (y_ref, q_ref, acc_ref) in zip(blocks, refs):
            assert np.array_equal(q[m0:m1], q_ref), "%s rows %d:%d: int8 codes differ" % (what, m0, m1)
            assert np.array_equal(acc[m0:m1], acc_ref), "%s rows %d:%d: int32 accumulators differ" % (what, m0, m1)
            assert_y_close(y[m0:m1], y_ref, "%s rows %d:%d" % (what, m0, m1))
            clip += int((np.abs(q_ref.astype(np.int32)) >= 127).sum())
        if not full:
            # codes are cheap for the oracle: compare all of them even when the matmul is sampled
            assert np.array_equal(q, q_all), "%s: int8 codes differ" % what
    layer.close()
    return clip
