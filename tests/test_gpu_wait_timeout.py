"""The bounded device-side wait really gives up, reports it, and leaves the handle and the context usable.

The failure is made without faulting or hanging anything: a tiny kernel waits a few dozen microseconds on
a barrier that nothing signals and that no copy or tensor-core operation refers to, then returns."""
import numpy as np
import pytest

import oracle
from paper_2412_20386_b200 import workloads as wl
from parity_util import assert_y_close, layer_inputs

pytestmark = pytest.mark.gpu


def test_wait_that_nothing_ends_sets_the_status_word_and_the_layer_keeps_working():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import __graft_entry__ as entry
    entry.build()
    import paper_2412_20386_b200 as ptq
    torch.cuda.set_device(0)

    spec = wl.configs()[0][0]
    x, wq, dw, bias, s, dx = layer_inputs(spec, B=2)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    other = ptq.PtqLinear(wq, dw, s, dx, bias)        # a second handle: its status word must stay clean
    xd = torch.from_numpy(x).cuda()
    y0 = layer.forward(xd)
    torch.cuda.synchronize()
    layer.device_status()                              # clean before the self-test

    short, long_, waited_ns = layer.selftest_wait_timeout(limit_us=50)
    assert short == 0, "the short wait must give up"
    assert long_ == 0, "the second wait must leave through the CTA's abort flag"
    assert waited_ns < 100_000_000, "the abort flag must end the long wait at once, not after its own limit"
    with pytest.raises(ptq.PtqError) as e:
        layer.device_status()
    assert e.value.status == 8 and "bounded wait" in str(e.value)
    layer.device_status()                              # reading the word cleared it
    other.device_status()

    # the handle and the context still work, and the result still matches the oracle
    y1 = layer.forward(xd)
    torch.cuda.synchronize()
    layer.device_status()
    assert torch.equal(y0, y1)
    y_ref = oracle.linear_forward(x.reshape(-1, spec.K), spec.T, wq, dw, s, dx, bias)
    assert_y_close(y1.cpu().numpy().reshape(-1, spec.N), y_ref, "forward after the timeout self-test")

    L = ptq.load_library()
    import ctypes
    out = (ctypes.c_uint * 3)()
    assert L.ptq_linear_selftest_wait_timeout(layer._h, 0, out, None) == 3          # limit out of range
    assert L.ptq_linear_selftest_wait_timeout(None, 50, out, None) == 1
    layer.close()
    other.close()
