"""GPU parity tests of the step-size search (Sec. 5.2, second stage): every loss against the oracle's
(binary64 sums in another order: 1e-12 relative), the chosen candidate equal to the oracle's wherever
the oracle's two best losses are further apart than that, the chosen step bit for bit, and a layer
built on the searched steps against the oracle end to end."""
import numpy as np
import pytest

import oracle
from paper_2412_20386_b200 import workloads as wl
from parity_util import assert_y_close

pytestmark = pytest.mark.gpu

CFG = wl.configs()
F32 = np.float32


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


def check_search(ptq, torch, xcal, s, base, n_grid, j_lo):
    dx, best, loss = ptq.search_act_step(torch.from_numpy(xcal).cuda(), s, base, n_grid, j_lo, want_loss=True)
    dx_ref, best_ref, loss_ref = oracle.search_act_step(xcal, s, base, n_grid, j_lo)
    assert loss.shape == loss_ref.shape
    assert np.all(np.abs(loss - loss_ref) <= 1e-12 * np.maximum(loss_ref, 1e-300)), "losses differ"
    T = xcal.shape[1]
    rows = np.arange(T)
    # the GPU's choice is a minimiser of the oracle's losses up to the summation-order tolerance
    assert np.all(loss_ref[rows, best - j_lo] <= loss_ref.min(axis=1) * (1 + 1e-11))
    srt = np.sort(loss_ref, axis=1)
    clear = (srt[:, 1] - srt[:, 0] > 1e-9 * np.maximum(srt[:, 0], 1e-300)) if loss_ref.shape[1] > 1 else np.ones(T, bool)
    assert np.array_equal(best[clear], best_ref[clear])
    ratio = (best.astype(F32) / F32(n_grid)).astype(F32)
    assert np.array_equal(dx.view(np.uint32), (base * ratio).astype(F32).view(np.uint32))
    dx2, best2, none = ptq.search_act_step(torch.from_numpy(xcal).cuda(), s, base, n_grid, j_lo)
    assert none is None and np.array_equal(dx, dx2) and np.array_equal(best, best2)      # reproducible
    return dx, best, best_ref, clear


@pytest.mark.parametrize("cfg,idx", [(0, 0), (1, 0), (1, 2), (3, 1), (4, 7)])
def test_search_on_workload_calibration_batches(env, cfg, idx):
    ptq, torch = env
    spec = CFG[cfg][idx]
    xcal = wl.activations(spec, wl.ROLE_CALIB)
    wq, dw, _ = wl.weights(spec)
    s, base = oracle.calibrate(xcal, wq, dw)
    dx, best, best_ref, clear = check_search(ptq, torch, xcal, s, base, 100, 20)
    assert clear.mean() > 0.95 and np.array_equal(best, best_ref)
    if spec.K >= 192:
        assert (best < 100).mean() > 0.5          # heavy-tailed rows: truncation pays at most positions


def test_search_small_grids_ties_and_specials(env):
    ptq, torch = env
    rng = np.random.default_rng(2)
    # planted three-way ties (multiples of the full step, power-of-two base): the largest j must win
    base = np.array([2.0 ** -3, 2.0 ** -5], F32)
    m = np.arange(-15, 17).astype(np.float64)
    x = np.stack([m * base[0], m * base[1]])[None].astype(np.float16)
    dx, best, loss = ptq.search_act_step(torch.from_numpy(x).cuda(), np.ones(32, F32), base, 4, 1, want_loss=True)
    assert np.all(loss[:, [0, 1, 3]] == 0) and np.all(loss[:, 2] > 0) and best.tolist() == [4, 4]
    assert np.array_equal(dx, base)
    # a single candidate; a grid that is not a multiple of the candidates a block takes; j_lo = n_grid
    x = rng.standard_normal((3, 7, 40)).astype(np.float16)
    x[0, 1, 3] = np.inf
    x[1, 2, 5] = np.nan
    x[2, 3, :] = 0
    s = np.exp(rng.uniform(-1, 1, 40)).astype(F32)
    base = np.full(7, 0.05, F32)
    for n_grid, j_lo in ((1, 1), (13, 2), (100, 100), (64, 1)):
        check_search(ptq, torch, x, s, base, n_grid, j_lo)


def test_search_argument_errors(env):
    ptq, torch = env
    x = torch.zeros((2, 3, 8), dtype=torch.float16, device="cuda")
    s = np.ones(8, F32)
    base = np.ones(3, F32)
    for (n_grid, j_lo) in ((0, 0), (10, 0), (10, 11), (5000, 1)):
        with pytest.raises(ptq.PtqError) as e:
            ptq.search_act_step(x, s, base, n_grid, j_lo)
        assert e.value.status == 3
    bad = base.copy()
    bad[1] = 0.0
    with pytest.raises(ptq.PtqError) as e:
        ptq.search_act_step(x, s, bad)
    assert e.value.status == 3
    bad_s = s.copy()
    bad_s[2] = np.nan
    with pytest.raises(ptq.PtqError) as e:
        ptq.search_act_step(x, bad_s, base)
    assert e.value.status == 3


def test_layer_on_searched_steps_matches_oracle(env):
    """The searched steps clip on purpose: the forward pass saturates codes exactly as the oracle does."""
    ptq, torch = env
    spec = CFG[1][3]
    xcal = wl.activations(spec, wl.ROLE_CALIB)
    wq, dw, bias = wl.weights(spec)
    s, base = oracle.calibrate(xcal, wq, dw)
    dx, best, _ = ptq.search_act_step(torch.from_numpy(xcal).cuda(), s, base)
    x = wl.activations(spec, wl.ROLE_EVAL, B=4)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    y, q, acc = layer.forward_debug(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    layer.device_status()
    x2 = x.reshape(-1, spec.K)
    y_ref, q_ref, acc_ref = oracle.linear_forward(x2, spec.T, wq, dw, s, dx, bias, taps=True)
    assert np.array_equal(q.cpu().numpy().reshape(-1, spec.K), q_ref)
    assert np.array_equal(acc.cpu().numpy().reshape(-1, spec.N), acc_ref)
    assert_y_close(y.cpu().numpy().reshape(-1, spec.N), y_ref, "searched steps")
    assert (np.abs(q_ref.astype(np.int32)) >= 127).sum() > 100
    layer.close()
