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

    for xin in (x1, x2):
        want = layer.forward(xin)
        got = torch.full_like(want, float("nan"))
        layer.forward_static(xin, got)
        torch.cuda.synchronize()
        layer.device_status()
        assert_y_close(got.cpu().numpy(), want.cpu().numpy(), "forward_static vs forward")
        assert torch.equal(got, want)                 # same kernels, same codes: in fact bit-identical
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
