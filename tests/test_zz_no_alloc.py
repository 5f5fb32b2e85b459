"""The allocation-free entry point, ``ptq_linear_forward_static``.

It serves callers that are not allowed to allocate device memory (a serving loop that must stay
off the allocator, a host application whose memory pool owns the whole device, a plugin that only
receives its input and output buffers): the int8 codes go to a scratch array built into the
library instead of a caller workspace.  This test calls it through the C ABI twice in a row, with
different inputs, and requires the same output as ``ptq_linear_forward`` -- the second call proves
that whatever the first one left in the shared scratch does no harm.  It lives in a file that
pytest collects last, so a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

import oracle
from paper_2412_20386_b200 import workloads as wl
from parity_util import assert_y_close, layer_inputs

pytestmark = pytest.mark.gpu


def test_forward_static_matches_forward_on_two_calls_in_a_row():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import __graft_entry__ as entry
    entry.build()
    import paper_2412_20386_b200 as ptq
    torch.cuda.set_device(0)

    spec = wl.configs()[2][1].with_batch(40)          # Vim-S out_proj 768 -> 384, 7880 rows, 6 MB of codes
    x, wq, dw, bias, s, dx = layer_inputs(spec)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    x1 = torch.from_numpy(x).cuda()
    x2 = torch.flip(x1, dims=[0]).contiguous()        # same layer, different batch content
    # a smaller call in between leaves stale bytes of another shape in the scratch
    small = wl.configs()[0][0]
    xs, wqs, dws, biass, ss, dxs = layer_inputs(small, B=2)
    layer_s = ptq.PtqLinear(wqs, dws, ss, dxs, biass)
    xsd = torch.from_numpy(xs).cuda()

    x_np = {id(x1): x, id(x2): x[::-1]}
    for xin in (x1, x2):
        want = layer.forward(xin)
        got = torch.full_like(want, float("nan"))
        layer.forward_static(xin, got)
        torch.cuda.synchronize()
        layer.device_status()
        assert_y_close(got.cpu().numpy(), want.cpu().numpy(), "forward_static vs forward")
        assert torch.equal(got, want)                 # same kernels, same codes: in fact bit-identical
        y_ref = oracle.linear_forward(np.ascontiguousarray(x_np[id(xin)]).reshape(-1, spec.K), spec.T, wq, dw, s, dx, bias)
        assert_y_close(got.cpu().numpy().reshape(-1, spec.N), y_ref, "forward_static vs oracle")
        ys = torch.empty((2, small.T, small.N), dtype=torch.float16, device="cuda")
        layer_s.forward_static(xsd, ys)
        assert torch.equal(ys, layer_s.forward(xsd))

    # a batch whose codes do not fit the built-in scratch is refused with a clear error
    big_B = ptq.binding.STATIC_SCRATCH_BYTES // (spec.T * layer.code_pitch()) + 1
    xb = torch.zeros((big_B, spec.T, spec.K), dtype=torch.float16, device="cuda")
    yb = torch.empty((big_B, spec.T, spec.N), dtype=torch.float16, device="cuda")
    with pytest.raises(ptq.PtqError) as e:
        layer.forward_static(xb, yb)
    assert e.value.status == 2 and "scratch" in str(e.value)


def test_forward_static_back_to_back_without_syncs_and_other_layer_kinds():
    """The supported usage: calls queued one after another on ONE stream, with no host synchronisation in
    between, all sharing the built-in scratch.  The quantize kernel of call i+1 may be scheduled while the
    GEMM of call i still runs; stream order must still hold for the shared array.  Symmetric, asymmetric and
    W4A4 handles alternate, and every output is compared with the CPU oracle afterwards."""
    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2412_20386_b200 as ptq
    torch.cuda.set_device(0)

    spec_a = wl.configs()[1][0]                        # in_proj 192 -> 768
    spec_b = wl.configs()[1][3]                        # out_proj 384 -> 192
    B = 16
    xa, wqa, dwa, ba, sa, dxa = layer_inputs(spec_a, B=B)
    xb, wqb, dwb, bb, sb, dxb = layer_inputs(spec_b, B=B)
    la = ptq.PtqLinear(wqa, dwa, sa, dxa, ba)
    s_as, dx_as, z_as = oracle.calibrate_asym(wl.activations(spec_b, wl.ROLE_CALIB), wqb, dwb)
    lb = ptq.PtqLinear(wqb, dwb, s_as, dx_as, bb, act_zero=z_as)
    w4 = np.clip(np.rint(wqa.astype(np.float32) / 18.0), -8, 7).astype(np.int8)
    s4, dx4 = oracle.calibrate4(wl.activations(spec_a, wl.ROLE_CALIB), w4, dwa)
    lc = ptq.PtqLinear(oracle.pack_int4(w4), dwa, s4, dx4, ba, packed4_K=spec_a.K)

    xad, xbd = torch.from_numpy(xa).cuda(), torch.from_numpy(xb).cuda()
    rounds = 12
    ya = [torch.empty((B, spec_a.T, spec_a.N), dtype=torch.float16, device="cuda") for _ in range(rounds)]
    yb = [torch.empty((B, spec_b.T, spec_b.N), dtype=torch.float16, device="cuda") for _ in range(rounds)]
    yc = [torch.empty((B, spec_a.T, spec_a.N), dtype=torch.float16, device="cuda") for _ in range(rounds)]
    torch.cuda.synchronize()
    for i in range(rounds):                            # 36 calls, no synchronisation in between
        la.forward_static(xad, ya[i])
        lb.forward_static(xbd, yb[i])
        lc.forward_static(xad, yc[i])
    torch.cuda.synchronize()
    for layer in (la, lb, lc):
        layer.device_status()
    ra = oracle.linear_forward(xa.reshape(-1, spec_a.K), spec_a.T, wqa, dwa, sa, dxa, ba)
    rb = oracle.linear_forward_asym(xb.reshape(-1, spec_b.K), spec_b.T, wqb, dwb, s_as, dx_as, z_as, bb)
    rc = oracle.linear_forward4(xa.reshape(-1, spec_a.K), spec_a.T, w4, dwa, s4, dx4, ba)
    for i in range(rounds):
        assert torch.equal(ya[i], ya[0]) and torch.equal(yb[i], yb[0]) and torch.equal(yc[i], yc[0])
    assert_y_close(ya[0].cpu().numpy().reshape(-1, spec_a.N), ra, "static, symmetric layer vs oracle")
    assert_y_close(yb[0].cpu().numpy().reshape(-1, spec_b.N), rb, "static, asymmetric layer vs oracle")
    assert_y_close(yc[0].cpu().numpy().reshape(-1, spec_a.N), rc, "static, W4A4 layer vs oracle")
