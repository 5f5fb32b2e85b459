"""GPU parity of the per-tensor static comparator (latency table of Sec. 6, Fig. 5): one activation step
for the whole tensor.  It is a PTS layer whose steps are all equal, so it runs the same kernels; what is
checked here is the calibration entry point against the oracle's, and a layer built from its result
against the oracle on every row."""
import numpy as np
import pytest

import oracle
from paper_2412_20386_b200 import workloads as wl
from parity_util import assert_y_close, row_blocks

pytestmark = pytest.mark.gpu

CFG = wl.configs()


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import __graft_entry__ as entry
    entry.build()
    import paper_2412_20386_b200 as ptq
    ptq.load_library()
    torch.cuda.set_device(0)
    return ptq, torch


@pytest.mark.parametrize("cfg,idx", [(0, 0), (1, 0), (1, 2), (1, 3), (2, 1)])
def test_per_tensor_static_layer(env, cfg, idx):
    ptq, torch = env
    spec = CFG[cfg][idx]
    x = wl.activations(spec, wl.ROLE_EVAL)
    xcal = wl.activations(spec, wl.ROLE_CALIB)
    wq, dw, bias = wl.weights(spec)
    s_ref, delta = oracle.calibrate_per_tensor(xcal, wq, dw)
    s, dx = ptq.calibrate(torch.from_numpy(xcal).cuda(), wq, dw, per_tensor=True)
    assert np.array_equal(s.view(np.uint32), s_ref.view(np.uint32))
    assert dx.shape == (spec.T,) and np.all(dx.view(np.uint32) == np.float32(delta).view(np.uint32))
    _, dx_pts = oracle.calibrate(xcal, wq, dw)
    assert delta == dx_pts.max()

    M = x.shape[0] * spec.T
    x2 = x.reshape(M, spec.K)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xd = torch.from_numpy(x).cuda()
    for flags in (0, ptq.FLAG_FUSED_PROLOGUE):
        y, q, acc = layer.forward_debug(xd, flags=flags)
        torch.cuda.synchronize()
        layer.device_status()
        y = y.cpu().numpy().reshape(M, spec.N)
        q = q.cpu().numpy().reshape(M, spec.K)
        acc = acc.cpu().numpy().reshape(M, spec.N)
        for (m0, m1) in row_blocks(M):
            y_ref, q_ref, acc_ref = oracle.linear_forward(x2, spec.T, wq, dw, s_ref, dx, bias, rows=(m0, m1), taps=True)
            assert np.array_equal(q[m0:m1], q_ref) and np.array_equal(acc[m0:m1], acc_ref)
            assert_y_close(y[m0:m1], y_ref, "%s per-tensor rows %d:%d" % (spec.name, m0, m1))
    layer.close()


def test_per_tensor_degenerate_batch_gives_the_floor(env):
    ptq, torch = env
    xcal = torch.zeros((2, 5, 16), dtype=torch.float16, device="cuda")
    s, dx = ptq.calibrate(xcal, np.ones((4, 16), np.int8), np.full(4, 0.01, np.float32), per_tensor=True)
    assert np.all(dx == np.float32(np.float32(1e-5) / np.float32(127)))
    s_ref, d_ref = oracle.calibrate_per_tensor(xcal.cpu().numpy(), np.ones((4, 16), np.int8), np.full(4, 0.01, np.float32))
    assert np.array_equal(s, s_ref) and dx[0] == d_ref
