"""GPU parity tests of the asymmetric PTS layer (step and zero offset per token position, Sec. 5.1 with
the quantizer form of Sec. 2.3): unsigned codes and offset-free int32 accumulators bit for bit against
the oracle, fp16 outputs within max(2^-10 |ref|, 1e-3)."""
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


def skewed(spec, role, B=None):
    """The workload's activations shifted and one-sided in places, so that the zero offsets spread over
    [0, 255] instead of sitting at 128."""
    x = wl.activations(spec, role, B=B).astype(np.float32)
    g, _ = wl.structure(spec)
    shift = (0.75 * g * np.cos(np.arange(spec.T)))[None, :, None]
    x = x + shift
    x[:, ::7, :] = np.abs(x[:, ::7, :])              # every 7th position is non-negative: offset 0
    return np.clip(x, -65504, 65504).astype(np.float16)


def check_asym(ptq, torch, spec, B=None):
    x = skewed(spec, wl.ROLE_EVAL, B)
    wq, dw, bias = wl.weights(spec)
    s, dx, z = oracle.calibrate_asym(skewed(spec, wl.ROLE_CALIB), wq, dw)
    Bn = x.shape[0]
    M = Bn * spec.T
    layer = ptq.PtqLinear(wq, dw, s, dx, bias, act_zero=z)
    assert not layer.fused_supported() and "asymmetric" in layer.describe()
    xd = torch.from_numpy(x).cuda()
    x2 = x.reshape(M, spec.K)
    blocks = row_blocks(M)                       # every row, one block at a time
    for flags in (0, ptq.FLAG_FUSED_PROLOGUE | ptq.FLAG_CTA_PAIR):      # the flags are accepted and ignored
        y, c, acc = layer.forward_debug(xd, flags=flags)
        y2 = layer.forward(xd, flags=flags)
        torch.cuda.synchronize()
        layer.device_status()
        assert torch.equal(y, y2) and c.dtype == torch.uint8
        y = y.cpu().numpy().reshape(M, spec.N)
        c = c.cpu().numpy().reshape(M, spec.K)
        acc = acc.cpu().numpy().reshape(M, spec.N)
        for (m0, m1) in blocks:
            y_ref, c_ref, acc_ref = oracle.linear_forward_asym(x2, spec.T, wq, dw, s, dx, z, bias, rows=(m0, m1), taps=True)
            assert np.array_equal(c[m0:m1], c_ref), "%s rows %d:%d: codes differ" % (spec.name, m0, m1)
            assert np.array_equal(acc[m0:m1], acc_ref), "%s rows %d:%d: accumulators differ" % (spec.name, m0, m1)
            assert_y_close(y[m0:m1], y_ref, "%s rows %d:%d" % (spec.name, m0, m1))
    assert len(np.unique(z)) > 8 and z.min() == 0                      # the offsets really vary
    layer.close()


def test_asym_config0(env):
    check_asym(*env, CFG[0][0])


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_asym_config1_block_linears(env, idx):
    check_asym(*env, CFG[1][idx])


@pytest.mark.parametrize("cfg,idx", [(2, 0), (3, 1), (4, 0), (4, 7)])
def test_asym_large_layers_every_row(env, cfg, idx):
    check_asym(*env, CFG[cfg][idx])


def test_asym_quantizer_all_fp16_inputs_and_tie_adjacent(env):
    ptq, torch = env
    rng = np.random.default_rng(41)
    for (T, K) in ((8, 64), (5, 12)):
        s = np.exp(rng.uniform(np.log(2e-3), np.log(3e2), K)).astype(np.float32)
        dx = np.exp(rng.uniform(np.log(1e-3), np.log(1e1), T)).astype(np.float32)
        z = rng.integers(0, 256, T).astype(np.int32)
        z[0], z[1] = 0, 255
        B = 65536
        base = (np.arange(B * T, dtype=np.int64) // T).astype(np.uint16)
        x = (np.repeat(base[:, None], K, axis=1) + (np.arange(K, dtype=np.uint16) * 977)[None, :]).astype(np.uint16)
        xh = x.view(np.float16).reshape(B, T, K)
        layer = ptq.PtqLinear(np.ones((4, K), np.int8), np.ones(4, np.float32), s, dx, act_zero=z)
        c = layer.quantize(torch.from_numpy(xh).cuda()).cpu().numpy().reshape(-1, K)
        assert np.array_equal(c, oracle.quantize_asym(xh.reshape(-1, K), T, s, dx, z))
    # tie-adjacent inputs over the whole signed range of round(v): -255.5 .. 255.5
    T, K, N = 16, 64, 16
    s = np.exp(rng.uniform(np.log(5e-2), np.log(2e1), K)).astype(np.float32)
    dx = np.exp(rng.uniform(np.log(1e-2), np.log(1.0), T)).astype(np.float32)
    z = rng.integers(0, 256, T).astype(np.int32)
    j = (np.arange(512) - 256 + 0.5)
    x = (j[:, None, None] * (s.astype(np.float64)[None, None, :] * dx.astype(np.float64)[None, :, None]))
    x = np.clip(x, -65504, 65504).astype(np.float16)
    x = np.concatenate([x, np.nextafter(x, np.float16(np.inf)), np.nextafter(x, np.float16(-np.inf))], axis=0)
    wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
    layer = ptq.PtqLinear(wq, np.full(N, 0.01, np.float32), s, dx, act_zero=z)
    _, c, acc = layer.forward_debug(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    layer.device_status()
    c_ref = oracle.quantize_asym(x.reshape(-1, K), T, s, dx, z)
    assert np.array_equal(c.cpu().numpy().reshape(-1, K), c_ref)
    assert np.array_equal(acc.cpu().numpy().reshape(-1, N), oracle.int_matmul_asym(c_ref, z, T, wq))


def test_asym_calibration_kernels_match_oracle(env):
    ptq, torch = env
    for spec in (CFG[0][0], CFG[1][2], CFG[4][7]):
        xcal = skewed(spec, wl.ROLE_CALIB)
        wq, dw, _ = wl.weights(spec)
        s, dx, z = ptq.calibrate_asym(torch.from_numpy(xcal).cuda(), wq, dw)
        s_ref, dx_ref, z_ref = oracle.calibrate_asym(xcal, wq, dw)
        assert np.array_equal(s.view(np.uint32), s_ref.view(np.uint32))
        assert np.array_equal(dx.view(np.uint32), dx_ref.view(np.uint32))
        assert np.array_equal(z, z_ref)
    xcal = np.zeros((2, 3, 16), np.float16)
    xcal[:, 0, :] = 2.0
    xcal[:, 1, :] = -3.0
    wq = np.full((4, 16), 10, np.int8)
    dw = np.full(4, 0.1, np.float32)
    s, dx, z = ptq.calibrate_asym(torch.from_numpy(xcal).cuda(), wq, dw)
    s_ref, dx_ref, z_ref = oracle.calibrate_asym(xcal, wq, dw)
    assert np.array_equal(s, s_ref) and np.array_equal(dx, dx_ref) and np.array_equal(z, z_ref)
    assert z.tolist() == [0, 255, 0]


def test_asym_create_rejects_bad_offsets(env):
    ptq, torch = env
    K, N, T = 16, 8, 4
    args = (np.ones((N, K), np.int8), np.full(N, 0.01, np.float32), np.ones(K, np.float32), np.ones(T, np.float32))
    for bad in (-1, 256):
        z = np.zeros(T, np.int32)
        z[2] = bad
        with pytest.raises(ptq.PtqError) as e:
            ptq.PtqLinear(*args, act_zero=z)
        assert e.value.status == 3
