"""GPU parity tests of W4A4 layers (the bit width of the paper's latency table; packing of Appendix B.1):
4-bit codes, packed bytes and int32 accumulators bit for bit against the oracle, fp16 outputs within
max(2^-10 |ref|, 1e-3)."""
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


def weights4(spec):
    """4-bit weights for a workload layer: the seeded int8 weights divided down to [-7, 7]."""
    wq8, dw, bias = wl.weights(spec)
    w4 = np.clip(np.rint(wq8.astype(np.float32) / 18.0), -8, 7).astype(np.int8)
    return w4, oracle.pack_int4(w4), dw, bias


def check_w4a4(ptq, torch, spec, B=None):
    x = wl.activations(spec, wl.ROLE_EVAL, B=B)
    xcal = wl.activations(spec, wl.ROLE_CALIB)
    w4, packed, dw, bias = weights4(spec)
    s_ref, dx_ref = oracle.calibrate4(xcal, w4, dw)
    s, dx = ptq.calibrate_w4a4(torch.from_numpy(xcal).cuda(), packed, spec.K, dw)
    assert np.array_equal(s.view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(dx.view(np.uint32), dx_ref.view(np.uint32))
    M = x.shape[0] * spec.T
    layer = ptq.PtqLinear(packed, dw, s, dx, bias, packed4_K=spec.K)
    assert "w4a4" in layer.describe() and not layer.fused_supported()
    xd = torch.from_numpy(x).cuda()
    x2 = x.reshape(M, spec.K)
    q_ref = oracle.quantize4(x2, spec.T, s, dx)
    blocks = row_blocks(M)                       # every row, one block at a time
    for flags in (0, ptq.FLAG_FUSED_PROLOGUE | ptq.FLAG_CTA_PAIR):           # accepted and ignored
        y, q, acc = layer.forward_debug(xd, flags=flags)
        y2 = layer.forward(xd, flags=flags)
        torch.cuda.synchronize()
        layer.device_status()
        assert torch.equal(y, y2)
        q = q.cpu().numpy().reshape(M, spec.K)
        assert np.array_equal(q, q_ref), "%s: 4-bit codes differ" % spec.name
        y = y.cpu().numpy().reshape(M, spec.N)
        acc = acc.cpu().numpy().reshape(M, spec.N)
        for (m0, m1) in blocks:
            acc_ref = oracle.int_matmul(q_ref[m0:m1], w4)
            assert np.array_equal(acc[m0:m1], acc_ref), "%s rows %d:%d: accumulators differ" % (spec.name, m0, m1)
            t0 = m0 % spec.T
            dx_rows = np.resize(np.roll(dx, -t0), m1 - m0)
            y_ref = oracle.dequant(acc_ref, m1 - m0, dx_rows, dw, bias)
            assert_y_close(y[m0:m1], y_ref, "%s rows %d:%d" % (spec.name, m0, m1))
    packed_codes = layer.quantize_packed4(xd).cpu().numpy().reshape(M, -1)
    assert np.array_equal(packed_codes, oracle.pack_int4(q_ref)), "%s: packed codes differ" % spec.name
    assert q_ref.min() >= -8 and q_ref.max() == 7
    with pytest.raises(ptq.PtqError) as e:
        layer.forward_dynamic(xd)
    assert e.value.status == 3
    layer.close()


def test_w4a4_config0(env):
    check_w4a4(*env, CFG[0][0])
    check_w4a4(*env, CFG[0][0], B=5)


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_w4a4_config1_block_linears(env, idx):
    # K = 12 takes the generic quantize kernel; N = 44 the masked stores
    check_w4a4(*env, CFG[1][idx])


@pytest.mark.parametrize("cfg,idx", [(3, 0), (3, 1), (4, 1)])
def test_w4a4_large_layers_every_row(env, cfg, idx):
    check_w4a4(*env, CFG[cfg][idx])


def test_w4a4_quantizer_all_fp16_inputs_ties_and_odd_k(env):
    ptq, torch = env
    rng = np.random.default_rng(8)
    for (T, K) in ((8, 64), (5, 13)):
        s = np.exp(rng.uniform(np.log(2e-3), np.log(3e2), K)).astype(np.float32)
        dx = np.exp(rng.uniform(np.log(1e-2), np.log(1e2), T)).astype(np.float32)
        B = 65536
        base = (np.arange(B * T, dtype=np.int64) // T).astype(np.uint16)
        x = (np.repeat(base[:, None], K, axis=1) + (np.arange(K, dtype=np.uint16) * 977)[None, :]).astype(np.uint16)
        xh = x.view(np.float16).reshape(B, T, K)
        w4 = np.ones((4, K), np.int8)
        layer = ptq.PtqLinear(oracle.pack_int4(w4), np.ones(4, np.float32), s, dx, packed4_K=K)
        xd = torch.from_numpy(xh).cuda()
        q = layer.quantize(xd).cpu().numpy().reshape(-1, K)
        q_ref = oracle.quantize4(xh.reshape(-1, K), T, s, dx)
        assert np.array_equal(q, q_ref)
        assert np.array_equal(layer.quantize_packed4(xd).cpu().numpy().reshape(B * T, -1), oracle.pack_int4(q_ref))
        layer.close()
    # values on and next to every rounding tie of the 4-bit range
    T, K = 16, 64
    s = np.exp(rng.uniform(np.log(5e-2), np.log(2e1), K)).astype(np.float32)
    dx = np.exp(rng.uniform(np.log(1e-2), np.log(1.0), T)).astype(np.float32)
    j = (np.arange(40) - 20 + 0.5)
    x = (j[:, None, None] * (s.astype(np.float64)[None, None, :] * dx.astype(np.float64)[None, :, None]))
    x = np.clip(x, -65504, 65504).astype(np.float16)
    x = np.concatenate([x, np.nextafter(x, np.float16(np.inf)), np.nextafter(x, np.float16(-np.inf))], axis=0)
    layer = ptq.PtqLinear(oracle.pack_int4(np.ones((4, K), np.int8)), np.ones(4, np.float32), s, dx, packed4_K=K)
    q = layer.quantize(torch.from_numpy(x).cuda()).cpu().numpy().reshape(-1, K)
    assert np.array_equal(q, oracle.quantize4(x.reshape(-1, K), T, s, dx))
    layer.close()
