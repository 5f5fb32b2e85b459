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


def row_blocks(M, block=8192):
    """Contiguous row ranges that together cover every row; the oracle and the comparison work one block
    at a time so that host memory stays bounded on the largest layers."""
    return [(m0, min(M, m0 + block)) for m0 in range(0, M, block)]


def layer_inputs(spec, B=None):
    x = wl.activations(spec, wl.ROLE_EVAL, B=B)
    wq, dw, bias = wl.weights(spec)
    s, dx = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    return x, wq, dw, bias, s, dx


def check_layer(ptq, torch, spec, B=None, flags_list=(0, 1, 2), seed=0):
    """Forward with taps through the C ABI, once per entry of flags_list (0 = quantize kernel then
    GEMM kernel, 1 = PTQ_FLAG_FUSED_PROLOGUE, 2 = PTQ_FLAG_CTA_PAIR); compare the int8 codes and int32
    accumulators bit for bit and the fp16 output within tolerance on EVERY row of the layer."""
    x, wq, dw, bias, s, dx = layer_inputs(spec, B)
    Bn = x.shape[0]
    M = Bn * spec.T
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xd = torch.from_numpy(x).cuda()
    x2 = x.reshape(M, spec.K)
    blocks = row_blocks(M)
    refs = [oracle.linear_forward(x2, spec.T, wq, dw, s, dx, bias, rows=blk, taps=True) for blk in blocks]
    clip = sum(int((np.abs(q_ref.astype(np.int32)) >= 127).sum()) for _, q_ref, _ in refs)
    for flags in flags_list:
        what = "%s flags=%d" % (spec.name, flags)
        y, q, acc = layer.forward_debug(xd, flags=flags)
        y2 = layer.forward(xd, flags=flags)                   # the production entry point
        torch.cuda.synchronize()
        layer.device_status()
        assert torch.equal(y, y2), "%s: forward and forward_debug disagree" % what
        del y2
        y = y.cpu().numpy().reshape(M, spec.N)
        q = q.cpu().numpy().reshape(M, spec.K)
        acc = acc.cpu().numpy().reshape(M, spec.N)
        for (m0, m1), (y_ref, q_ref, acc_ref) in zip(blocks, refs):
            assert np.array_equal(q[m0:m1], q_ref), "%s rows %d:%d: int8 codes differ" % (what, m0, m1)
            assert np.array_equal(acc[m0:m1], acc_ref), "%s rows %d:%d: int32 accumulators differ" % (what, m0, m1)
            assert_y_close(y[m0:m1], y_ref, "%s rows %d:%d" % (what, m0, m1))
    layer.close()
    return clip
