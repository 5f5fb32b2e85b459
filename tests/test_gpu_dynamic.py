"""GPU parity tests of the per-token dynamic comparator (the alternative to PTS of Sec. 4.1 and the
latency table of Sec. 6): row steps and int8 codes and int32 accumulators bit for bit against the
oracle, fp16 outputs within max(2^-10 |ref|, 1e-3)."""
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


def check_dynamic(ptq, torch, spec, B=None, x=None):
    if x is None:
        x = wl.activations(spec, wl.ROLE_EVAL, B=B)
    wq, dw, bias = wl.weights(spec)
    s, dx = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    Bn = x.shape[0]
    M = Bn * spec.T
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xd = torch.from_numpy(x).cuda()
    x2 = x.reshape(M, spec.K)
    y, q, acc, step = layer.forward_dynamic_debug(xd)
    y2 = layer.forward_dynamic(xd)
    torch.cuda.synchronize()
    layer.device_status()
    assert torch.equal(y, y2) or (torch.equal(torch.isnan(y), torch.isnan(y2)) and
                                  torch.equal(torch.nan_to_num(y), torch.nan_to_num(y2)))
    y = y.cpu().numpy().reshape(M, spec.N)
    q = q.cpu().numpy().reshape(M, spec.K)
    acc = acc.cpu().numpy().reshape(M, spec.N)
    step = step.cpu().numpy()
    q_ref, step_ref = oracle.quantize_dynamic(x2, s)
    assert np.array_equal(step.view(np.uint32), step_ref.view(np.uint32)), "%s: row steps differ" % spec.name
    assert np.array_equal(q, q_ref), "%s: int8 codes differ" % spec.name
    blocks = row_blocks(M)                       # every row, one block at a time
    for (m0, m1) in blocks:
        acc_ref = oracle.int_matmul(q_ref[m0:m1], wq)
        assert np.array_equal(acc[m0:m1], acc_ref), "%s rows %d:%d: accumulators differ" % (spec.name, m0, m1)
        y_ref = oracle.dequant(acc_ref, m1 - m0, step_ref[m0:m1], dw, bias)
        finite = np.isfinite(step_ref[m0:m1])
        assert_y_close(y[m0:m1][finite], y_ref[finite], "%s rows %d:%d" % (spec.name, m0, m1))
    layer.close()
    return q_ref, step_ref


def test_dynamic_config0(env):
    check_dynamic(*env, CFG[0][0])
    check_dynamic(*env, CFG[0][0], B=5)          # 985 rows: not a multiple of the rows a warp or a CTA takes


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_dynamic_config1_block_linears(env, idx):
    # K = 192, 384, 12 (generic kernel: K % 8 != 0) and 384
    check_dynamic(*env, CFG[1][idx])


@pytest.mark.parametrize("cfg,idx", [(2, 1), (3, 0), (3, 1), (4, 0)])
def test_dynamic_large_layers_every_row(env, cfg, idx):
    check_dynamic(*env, CFG[cfg][idx])


def test_dynamic_special_rows(env):
    """Dead rows (floored step), rows holding inf / NaN, rows of denormals, a row at the fp16 maximum."""
    ptq, torch = env
    spec = CFG[0][0]
    x = wl.activations(spec, wl.ROLE_EVAL, B=4).copy()
    x[0, 3] = 0
    x[0, 4, 7] = np.inf
    x[0, 5, 9] = -np.inf
    x[0, 6, 11] = np.nan
    x[0, 7, :] = np.nan
    x[0, 8] = np.float16(6e-8)
    x[0, 9] = np.float16(65504)
    x[0, 10, ::2] = np.float16(-65504)
    x[1, 0, :] = 0
    x[1, 0, 383] = np.float16(1.0)                # the only live element is the last one of the row
    q_ref, step_ref = check_dynamic(ptq, torch, spec, x=x)
    assert np.isinf(step_ref[4]) and np.isinf(step_ref[5]) and np.isfinite(step_ref[6])
    assert step_ref[3] == step_ref[7] == np.float32(np.float32(1e-5) / np.float32(127))
    assert q_ref[spec.T + 0, 383] == 127


def test_dynamic_tie_adjacent_rows(env):
    """Rows built so that many elements sit on or next to a rounding tie of u / step."""
    ptq, torch = env
    rng = np.random.default_rng(77)
    T, K, N = 64, 256, 32
    s = np.exp(rng.uniform(np.log(5e-2), np.log(2e1), K)).astype(np.float32)
    # one anchor element per row fixes the step near a chosen value; the rest are half-integers times s * step
    step_target = np.exp(rng.uniform(np.log(1e-2), np.log(1.0), (6, T))).astype(np.float64)
    j = rng.integers(-126, 127, (6, T, K)) + 0.5
    x = j * s.astype(np.float64)[None, None, :] * step_target[:, :, None]
    x[:, :, 0] = 127.0 * s[0] * step_target
    x = np.clip(x, -65504, 65504).astype(np.float16)
    x = np.concatenate([x, np.nextafter(x, np.float16(np.inf)), np.nextafter(x, np.float16(-np.inf))], axis=0)
    wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
    layer = ptq.PtqLinear(wq, np.full(N, 0.01, np.float32), s, np.ones(T, np.float32))
    _, q, acc, step = layer.forward_dynamic_debug(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    layer.device_status()
    q_ref, step_ref = oracle.quantize_dynamic(x.reshape(-1, K), s)
    assert np.array_equal(step.cpu().numpy().view(np.uint32), step_ref.view(np.uint32))
    assert np.array_equal(q.cpu().numpy().reshape(-1, K), q_ref)
    assert np.array_equal(acc.cpu().numpy().reshape(-1, N), oracle.int_matmul(q_ref, wq))
    # the construction does put many values next to a tie
    u = (x.reshape(-1, K).astype(np.float32) / s[None, :]) / step_ref[:, None]
    assert (np.abs(np.abs(u - np.floor(u)) - 0.5) < 1e-2).sum() > 10000
    layer.close()


def test_dynamic_scales_outside_the_reciprocal_range_and_unaligned(env):
    ptq, torch = env
    rng = np.random.default_rng(5)
    T, K, N = 7, 40, 24
    wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
    dw = np.full(N, 0.02, np.float32)
    x = rng.standard_normal((3, T, K)).astype(np.float16)
    for s in (np.full(K, 1e-12, np.float32), np.full(K, 3e11, np.float32),
              np.exp(rng.uniform(-3, 3, K)).astype(np.float32)):
        layer = ptq.PtqLinear(wq, dw, s, np.ones(T, np.float32))
        # aligned, then x at an address that is 2 (mod 16): the generic kernel
        big = torch.zeros(3 * T * K + 8, dtype=torch.float16, device="cuda")
        for off in (0, 1):
            xd = big[off:off + 3 * T * K].view(3, T, K)
            xd.copy_(torch.from_numpy(x))
            _, q, acc, step = layer.forward_dynamic_debug(xd)
            torch.cuda.synchronize()
            layer.device_status()
            q_ref, step_ref = oracle.quantize_dynamic(x.reshape(-1, K), s)
            assert np.array_equal(step.cpu().numpy().view(np.uint32), step_ref.view(np.uint32))
            assert np.array_equal(q.cpu().numpy().reshape(-1, K), q_ref)
            assert np.array_equal(acc.cpu().numpy().reshape(-1, N), oracle.int_matmul(q_ref, wq))
        layer.close()


def test_dynamic_argument_errors(env):
    ptq, torch = env
    K, N, T = 16, 8, 4
    args = (np.ones((N, K), np.int8), np.full(N, 0.01, np.float32), np.ones(K, np.float32), np.ones(T, np.float32))
    x = torch.zeros((2, T, K), dtype=torch.float16, device="cuda")
    layer = ptq.PtqLinear(*args)
    assert layer.workspace_bytes_dynamic(2) == 256 + 2 * T * 4
    with pytest.raises(ptq.PtqError) as e:
        layer.forward_dynamic(x, workspace=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 2
    layer.close()
    asym = ptq.PtqLinear(*args, act_zero=np.zeros(T, np.int32))
    with pytest.raises(ptq.PtqError) as e:
        asym.forward_dynamic(x)
    assert e.value.status == 3
    asym.close()
