"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  int8 codes and int32 accumulators must match bit for bit; fp16 outputs within
max(2^-10 |ref|, 1e-3)."""
import numpy as np
import pytest

import oracle
from paper_2412_20386_b200 import workloads as wl
from parity_util import assert_y_close, check_layer, layer_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import __graft_entry__ as entry
    entry.build()
    import paper_2412_20386_b200 as ptq
    ptq.load_library()          # raises if the CUDA library is missing: there is no fallback
    torch.cuda.set_device(0)
    return ptq, torch


CFG = wl.configs()


def test_config0_vim_ti_out_proj_single_image(env):
    ptq, torch = env
    check_layer(ptq, torch, CFG[0][0])


C1_ALL_PATHS = [0, 1, 2, 3, 4 * 23 + 0, 4 * 11 + 1, 4 * 7 + 2, 4 * 17 + 3]


@pytest.mark.parametrize("idx", C1_ALL_PATHS)
def test_config1_vim_ti_block_linears_batch64(env, idx):
    ptq, torch = env
    clip = check_layer(ptq, torch, CFG[1][idx])
    assert clip > 0      # heavy tails beyond the calibration range do clip


@pytest.mark.parametrize("block", range(24))
def test_config1_every_layer_default_path(env, block):
    # all 96 linears of the 24 blocks through the default path (the eight above also take the fused and
    # CTA-pair flags)
    ptq, torch = env
    for idx in range(4 * block, 4 * block + 4):
        if idx not in C1_ALL_PATHS:
            check_layer(ptq, torch, CFG[1][idx], flags_list=(0,))


@pytest.mark.parametrize("idx", [0, 1])
def test_config2_vim_s_batch128(env, idx):
    ptq, torch = env
    check_layer(ptq, torch, CFG[2][idx])


@pytest.mark.parametrize("idx", [0, 1])
def test_config3_vim_b_batch256(env, idx):
    ptq, torch = env
    check_layer(ptq, torch, CFG[3][idx])


@pytest.mark.parametrize("idx", range(8))
def test_config4_vmamba_stages_batch64(env, idx):
    ptq, torch = env
    check_layer(ptq, torch, CFG[4][idx])


def test_quantizer_all_fp16_inputs_many_scales(env):
    # every binary16 bit pattern against 8 token steps x 64 channel scales (vector kernel), and against
    # 5 x 12 (scalar kernel); this is also the check of the reciprocal + FMA division route.
    ptq, torch = env
    rng = np.random.default_rng(11)
    for (T, K) in ((8, 64), (5, 12)):
        s = np.exp(rng.uniform(np.log(2e-3), np.log(3e2), K)).astype(np.float32)
        dx = np.exp(rng.uniform(np.log(1e-3), np.log(1e1), T)).astype(np.float32)
        s[0], dx[0] = 1.0, 1.0
        s[1], dx[1] = 3.0, 1.0 / 3.0
        B = 65536
        M = B * T
        base = (np.arange(M, dtype=np.int64) // T).astype(np.uint16)              # image b carries pattern b
        x = np.repeat(base[:, None], K, axis=1)
        x = (x + (np.arange(K, dtype=np.uint16) * 977)[None, :]).astype(np.uint16)   # every channel sees all patterns
        xh = x.view(np.float16).reshape(B, T, K)
        wq = np.ones((4, K), np.int8)
        layer = ptq.PtqLinear(wq, np.ones(4, np.float32), s, dx)
        q = layer.quantize(torch.from_numpy(xh).cuda()).cpu().numpy().reshape(M, K)
        want = oracle.quantize(xh.reshape(M, K), T, s, dx)
        assert np.array_equal(q, want)


def test_quantizer_tie_adjacent_inputs_all_paths(env):
    # x = fp16((j + 0.5) s[k] dx[t]) for every half-integer j + 0.5 in [-127.5, 127.5]: the quotient lands
    # within fp16 rounding of a tie, so thousands of elements (30 times the natural share) fall inside the screening band and
    # are decided by the exact two-division route.  Checked for the quantize kernel and, through the
    # accumulators, for the fused kernel's in-kernel quantizers.
    ptq, torch = env
    rng = np.random.default_rng(14)
    T, K, N = 16, 64, 16
    s = np.exp(rng.uniform(np.log(5e-2), np.log(2e1), K)).astype(np.float32)
    dx = np.exp(rng.uniform(np.log(1e-2), np.log(1.0), T)).astype(np.float32)
    j = (np.arange(256) - 128 + 0.5)
    x = (j[:, None, None] * (s.astype(np.float64)[None, None, :] * dx.astype(np.float64)[None, :, None])).astype(np.float16)
    x = np.concatenate([x, np.nextafter(x, np.float16(np.inf)), np.nextafter(x, np.float16(-np.inf))], axis=0)
    B = x.shape[0]
    wq = rng.integers(-127, 128, (N, K)).astype(np.int8)
    layer = ptq.PtqLinear(wq, np.full(N, 0.01, np.float32), s, dx)
    xd = torch.from_numpy(x).cuda()
    q_ref = oracle.quantize(x.reshape(-1, K), T, s, dx)
    q = layer.quantize(xd).cpu().numpy().reshape(-1, K)
    assert np.array_equal(q, q_ref)
    acc_ref = oracle.int_matmul(q_ref, wq)
    for flags in (0, ptq.FLAG_FUSED_PROLOGUE):
        _, q2, acc = layer.forward_debug(xd, flags=flags)
        torch.cuda.synchronize()
        layer.device_status()
        assert np.array_equal(q2.cpu().numpy().reshape(-1, K), q_ref)
        assert np.array_equal(acc.cpu().numpy().reshape(B * T, N), acc_ref)
    # how many elements actually sat inside the band (exact quotient within 6e-5 of a tie)
    v = x.astype(np.float64) / s.astype(np.float64)[None, None, :] / dx.astype(np.float64)[None, :, None]
    inside = np.abs(np.abs(v - np.floor(v)) - 0.5) < 6e-5
    assert inside.sum() > 1000


def test_forward_edge_arguments(env):
    ptq, torch = env
    spec = CFG[0][0]
    x, wq, dw, bias, s, dx = layer_inputs(spec, B=1)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    L = ptq.load_library()
    xd = torch.from_numpy(x).cuda()
    y = torch.empty((1, spec.T, spec.N), dtype=torch.float16, device="cuda")
    ws = torch.empty(layer.workspace_bytes(1), dtype=torch.uint8, device="cuda")
    for B in (0, -3):                                  # an empty batch is refused, nothing is launched
        n0 = ptq.binding.kernel_launch_count()
        assert L.ptq_linear_forward(layer._h, xd.data_ptr(), B, y.data_ptr(), ws.data_ptr(), ws.numel(), 0, None) == 2
        assert L.ptq_quantize(layer._h, xd.data_ptr(), B, ws.data_ptr(), None) == 2
        assert ptq.binding.kernel_launch_count() == n0
    assert layer.workspace_bytes(0) == 0
    assert L.ptq_linear_forward(layer._h, xd.data_ptr(), 1, xd.data_ptr(), ws.data_ptr(), ws.numel(), 0, None) == 3   # y aliases x
    assert L.ptq_linear_forward(layer._h, xd.data_ptr(), 1, y.data_ptr(), ws.data_ptr() + 8, ws.numel() - 8, 0, None) in (2, 4)
    assert "K=384 N=192" in layer.describe()


@pytest.mark.parametrize("K,N,T,B", [(16, 65536, 3, 3), (8, 24, 100003, 1), (8192, 8, 1, 300)])
def test_maximum_sizes(env, K, N, T, B):
    ptq, torch = env
    spec = wl.LinearSpec(8, 1, 1, "max", B, T, K, N, bias=True, n_outliers=1)
    check_layer(ptq, torch, spec)


def test_quantizer_scales_outside_reciprocal_range_use_ieee_division(env):
    ptq, torch = env
    rng = np.random.default_rng(12)
    T, K, B = 3, 32, 700
    s = np.exp(rng.uniform(-2, 2, K)).astype(np.float32)
    dx = np.exp(rng.uniform(-2, 2, T)).astype(np.float32)
    s[5] = 1e-12
    s[6] = 3e13
    dx[1] = 2e-11
    x = (rng.standard_normal((B, T, K)) * 10.0 ** rng.uniform(-7, 4, (B, T, K))).astype(np.float16)
    layer = ptq.PtqLinear(np.ones((4, K), np.int8), np.ones(4, np.float32), s, dx)
    q = layer.quantize(torch.from_numpy(x).cuda()).cpu().numpy().reshape(-1, K)
    assert np.array_equal(q, oracle.quantize(x.reshape(-1, K), T, s, dx))


def test_closed_form_integer_inputs_on_gpu(env):
    # s = dx = dw = 1 and integer-valued activations: codes equal the inputs and the output is the
    # exact integer matmul rounded to fp16 (checked against numpy int64, not against the oracle).
    ptq, torch = env
    rng = np.random.default_rng(13)
    B, T, K, N = 5, 61, 160, 72
    xi = rng.integers(-128, 128, (B, T, K))
    wq = rng.integers(-2, 3, (N, K)).astype(np.int8)
    one = lambda n: np.ones(n, np.float32)
    layer = ptq.PtqLinear(wq, one(N), one(K), one(T))
    y, q, acc = layer.forward_debug(torch.from_numpy(xi.astype(np.float16)).cuda())
    exact = xi.reshape(-1, K) @ wq.astype(np.int64).T
    assert np.array_equal(q.cpu().numpy().reshape(-1, K).astype(np.int64), xi.reshape(-1, K))
    assert np.array_equal(acc.cpu().numpy().reshape(-1, N).astype(np.int64), exact)
    assert np.array_equal(y.cpu().numpy().reshape(-1, N).view(np.uint16),
                          exact.astype(np.float64).astype(np.float16).view(np.uint16))


@pytest.mark.parametrize("K,N,T,B", [(12, 384, 197, 2), (384, 44, 197, 3), (96, 8, 7, 40), (1536, 768, 49, 6),
                                     (40, 300, 3, 50), (8192, 16, 2, 70), (129, 257, 5, 30), (16, 1000, 1, 131)])
def test_odd_shapes_and_ragged_tiles(env, K, N, T, B):
    ptq, torch = env
    spec = wl.LinearSpec(9, K % 97, N % 5, "odd", B, T, K, N, bias=(N % 2 == 0))
    check_layer(ptq, torch, spec)


@pytest.mark.parametrize("K,N,T,B,variant", [(520, 600, 197, 257, 2),      # panel kernel: ragged K, N and M tails, 5 k-blocks
                                             (776, 1032, 64, 300, 0),     # 7 k-blocks: too deep for a panel, streaming
                                             (72, 520, 197, 140, 1)])     # two-team epilogue: ragged K and N, 3 N tiles
def test_ragged_shapes_through_the_panel_and_team_kernels(env, K, N, T, B, variant):
    """Shapes chosen so that the resident-panel kernel and the two-team epilogue (and, as a control, the streaming
    kernel at the same size) see tails in every dimension: K not a multiple of 128, N not a multiple of the tile
    width, B*T not a multiple of 128, an uneven last round of work units."""
    ptq, torch = env
    spec = wl.LinearSpec(10, K % 89, N % 7, "ragged", B, T, K, N, bias=False)
    x, wq, dw, bias, s, dx = layer_inputs(spec, B=1)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    assert layer.gemm_variant(B) == variant
    layer.close()
    check_layer(ptq, torch, spec, flags_list=(0,))


def test_two_host_threads_share_one_handle(env):
    """Two host threads call forward on ONE handle at the same time, each on its own stream with its own buffers
    (ctypes releases the interpreter lock during the call, so the library's per-handle caches and one-time set-up
    are really entered concurrently).  Every output must equal the single-threaded one bit for bit."""
    import threading
    ptq, torch = env
    spec = CFG[1][0]
    x, wq, dw, bias, s, dx = layer_inputs(spec, B=8)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xd = torch.from_numpy(x).cuda()
    want = layer.forward(xd)
    torch.cuda.synchronize()
    outs, errors = {}, []

    def worker(tid):
        try:
            torch.cuda.set_device(0)
            st = torch.cuda.Stream()
            xs = xd.clone()
            ys = [torch.empty_like(want) for _ in range(6)]          # more buffers than cache entries
            ws = torch.empty(layer.workspace_bytes(8), dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()
            for i in range(60):
                layer.forward(xs, y=ys[i % 6], workspace=ws, stream=st)
            st.synchronize()
            outs[tid] = ys
        except Exception as e:                                        # noqa: BLE001 (reported below)
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    layer.device_status()
    for ys in outs.values():
        for y in ys:
            assert torch.equal(y, want)


def test_seeded_random_shapes(env):
    """Sixteen seeded random (K, N, T, B): every kernel variant the shape and alignment select, every flag."""
    ptq, torch = env
    rng = np.random.default_rng(20241228)
    for i in range(16):
        K = int(rng.integers(1, 700))
        N = int(rng.integers(1, 600))
        T = int(rng.integers(1, 60))
        B = int(rng.integers(1, 12)) * int(rng.choice([1, 1, 7]))
        if i % 4 == 0:
            K = (K + 7) // 8 * 8                     # some shapes on the vector paths
            N = (N + 7) // 8 * 8
        spec = wl.LinearSpec(8, i, i % 4, "rand%d" % i, B, T, K, N, bias=bool(i & 1))
        check_layer(ptq, torch, spec)


def test_back_to_back_layers_sharing_one_workspace(env):
    """Kernels of consecutive calls overlap at their edges (programmatic dependent launch): two layers that
    alternate on ONE stream and ONE workspace must still see each other's kernels in stream order."""
    ptq, torch = env
    specs = [wl.LinearSpec(7, 0, 0, "a", 24, 197, 384, 768), wl.LinearSpec(7, 1, 3, "b", 24, 197, 768, 192, bias=True)]
    layers, xs, refs = [], [], []
    need = 0
    for sp in specs:
        x, wq, dw, bias, s, dx = layer_inputs(sp)
        layer = ptq.PtqLinear(wq, dw, s, dx, bias)
        xd = torch.from_numpy(x).cuda()
        ref = layer.forward(xd).clone()                 # its own workspace, nothing else in flight
        torch.cuda.synchronize()
        layers.append(layer)
        xs.append(xd)
        refs.append(ref)
        need = max(need, layer.workspace_bytes(sp.B, 0), layer.workspace_bytes_dynamic(sp.B))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    ys = [torch.empty_like(r) for r in refs]
    for it in range(25):
        for i in (0, 1):
            if it % 5 == 4:
                layers[i].forward_dynamic(xs[i], y=ys[i], workspace=ws)      # a different kernel pair in between
            layers[i].forward(xs[i], y=ys[i], workspace=ws)
        if it % 6 == 0:
            torch.cuda.synchronize()
            assert torch.equal(ys[0], refs[0]) and torch.equal(ys[1], refs[1]), "iteration %d" % it
    torch.cuda.synchronize()
    assert torch.equal(ys[0], refs[0]) and torch.equal(ys[1], refs[1])
    for layer in layers:
        layer.device_status()
        layer.close()


def test_fused_flag_is_reported_and_needs_no_workspace(env):
    ptq, torch = env
    for spec, want in ((CFG[3][0], True), (CFG[3][1], True), (CFG[1][2], False),
                       (wl.LinearSpec(9, 0, 0, "bigk", 2, 5, 4096, 64), False)):
        x, wq, dw, bias, s, dx = layer_inputs(spec, B=2)
        layer = ptq.PtqLinear(wq, dw, s, dx, bias)
        assert layer.fused_supported() == want
        if want:
            assert layer.workspace_bytes(2, ptq.FLAG_FUSED_PROLOGUE) == 0
            xd = torch.from_numpy(x).cuda()
            y = torch.empty((2, spec.T, spec.N), dtype=torch.float16, device="cuda")
            L = ptq.load_library()
            st = L.ptq_linear_forward(layer._h, xd.data_ptr(), 2, y.data_ptr(), None, 0, ptq.FLAG_FUSED_PROLOGUE, None)
            assert st == 0
            torch.cuda.synchronize()
            layer.device_status()
            y_ref = oracle.linear_forward(x.reshape(-1, spec.K), spec.T, wq, dw, s, dx, bias)
            assert_y_close(y.cpu().numpy().reshape(-1, spec.N), y_ref, "fused without workspace")
        else:
            assert layer.workspace_bytes(2, ptq.FLAG_FUSED_PROLOGUE) == layer.workspace_bytes(2, 0) > 0


def test_unaligned_pointers_take_the_generic_paths(env):
    ptq, torch = env
    spec = CFG[0][0]
    x, wq, dw, bias, s, dx = layer_inputs(spec, B=2)
    M = 2 * spec.T
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xbuf = torch.zeros(x.size + 8, dtype=torch.float16, device="cuda")
    ybuf = torch.zeros(M * spec.N + 8, dtype=torch.float16, device="cuda")
    xv = xbuf[1:1 + x.size].view(2, spec.T, spec.K)          # 2-byte aligned only
    yv = ybuf[1:1 + M * spec.N].view(2, spec.T, spec.N)
    xv.copy_(torch.from_numpy(x).cuda())
    y_ref = oracle.linear_forward(x.reshape(M, spec.K), spec.T, wq, dw, s, dx, bias)
    for flags in (0, ptq.FLAG_FUSED_PROLOGUE):       # the fused flag falls back: x is not 16-byte aligned
        yv.zero_()
        layer.forward(xv, y=yv, workspace=torch.empty(layer.workspace_bytes(2), dtype=torch.uint8, device="cuda"),
                      flags=flags)
        torch.cuda.synchronize()
        layer.device_status()
        assert_y_close(yv.cpu().numpy().reshape(M, spec.N), y_ref, "unaligned flags=%d" % flags)
    assert float(ybuf[0]) == 0.0 and float(ybuf[-7:].abs().max()) == 0.0     # nothing written outside y


def test_repeated_runs_are_bit_identical_and_stay_inside_y(env):
    ptq, torch = env
    spec = CFG[1][3]
    x, wq, dw, bias, s, dx = layer_inputs(spec, B=16)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xd = torch.from_numpy(x).cuda()
    M = 16 * spec.T
    guard = 4096
    ybuf = torch.full((M * spec.N + 2 * guard,), -7.0, dtype=torch.float16, device="cuda")
    yv = ybuf[guard:guard + M * spec.N].view(16, spec.T, spec.N)
    ws = torch.empty(layer.workspace_bytes(16) + 2 * guard, dtype=torch.uint8, device="cuda")
    first = None
    for i in range(12):
        layer.forward(xd, y=yv, workspace=ws[guard:guard + layer.workspace_bytes(16)],
                      flags=ptq.FLAG_FUSED_PROLOGUE if i % 2 else 0)     # both paths give the same bits
        cur = yv.clone()
        first = cur if first is None else first
        assert torch.equal(cur, first)
    layer.device_status()
    assert bool((ybuf[:guard] == -7.0).all()) and bool((ybuf[-guard:] == -7.0).all())


def test_calibration_kernels_match_oracle_bit_for_bit(env):
    ptq, torch = env
    for spec in (CFG[0][0], CFG[1][2], CFG[4][7], CFG[4][0].with_batch(2)):
        xcal = wl.activations(spec, wl.ROLE_CALIB, B=min(8, spec.B))
        wq, dw, _ = wl.weights(spec)
        s, dx = ptq.calibrate(torch.from_numpy(xcal).cuda(), wq, dw)
        s_ref, dx_ref = oracle.calibrate(xcal, wq, dw)
        assert np.array_equal(s.view(np.uint32), s_ref.view(np.uint32))
        assert np.array_equal(dx.view(np.uint32), dx_ref.view(np.uint32))
    # degenerate: dead channels and positions
    xcal = np.zeros((2, 3, 16), np.float16)
    xcal[:, 1, 2] = 3.0
    wq = np.zeros((4, 16), np.int8)
    wq[:, 2] = [10, -20, 5, 40]
    dw = np.array([0.01, 0.01, 0.02, 0.02], np.float32)
    s, dx = ptq.calibrate(torch.from_numpy(xcal).cuda(), wq, dw)
    s_ref, dx_ref = oracle.calibrate(xcal, wq, dw)
    assert np.array_equal(s, s_ref) and np.array_equal(dx, dx_ref)


def test_forward_argument_errors_return_codes(env):
    ptq, torch = env
    spec = CFG[0][0]
    x, wq, dw, bias, s, dx = layer_inputs(spec, B=1)
    layer = ptq.PtqLinear(wq, dw, s, dx, bias)
    xd = torch.from_numpy(x).cuda()
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(ptq.PtqError) as e:
        layer.forward(xd, workspace=small)
    assert e.value.status == 2
    with pytest.raises(ptq.PtqError) as e:
        layer.forward(xd, flags=64)
    assert e.value.status == 3
    y = layer.forward(xd)          # the handle still works after refused calls
    torch.cuda.synchronize()
    layer.device_status()
    assert_y_close(y.cpu().numpy().reshape(-1, spec.N),
                   oracle.linear_forward(x.reshape(-1, spec.K), spec.T, wq, dw, s, dx, bias), "after errors")


def test_gemm_kernel_selection_covers_all_three_variants(env):
    """The three GEMM kernels are all reached by the configured workloads (so the parity tests above compare each
    of them with the oracle): streaming for one-tile layers and long main loops, the two-team epilogue for short
    main loops with many tiles, the resident-panel kernel for the Vim-B in_proj."""
    ptq, torch = env
    want = {(0, 0): 0, (3, 0): 2, (3, 1): 0, (4, 0): 1, (4, 2): 1, (2, 0): 1, (2, 1): 0}
    for (cfg, idx), variant in want.items():
        spec = CFG[cfg][idx]
        x, wq, dw, bias, s, dx = layer_inputs(spec, B=1)
        layer = ptq.PtqLinear(wq, dw, s, dx, bias)
        assert layer.gemm_variant(spec.B) == variant, (spec.name, spec.M, spec.K, spec.N, layer.gemm_variant(spec.B))
        assert layer.gemm_variant(0) == -1


def test_probe_kernels_report_plausible_rates(env):
    """The measurement aids behind the roofline discussion: on a B200 a pure store stream and TMA stores in the
    epilogue's pattern both exceed 3 TB/s, operand stages arrive from L2 faster than the stores leave, and an empty
    kernel launches in microseconds.  Small buffers and bad arguments are refused, and nothing is left in flight."""
    ptq, torch = env
    P = ptq.binding
    buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    st16 = P.probe(P.PROBE_STORE16, buf, 5)
    tma = P.probe(P.PROBE_TMA_STORE, buf, 5)
    pull = P.probe(P.PROBE_OPERAND_PULL, buf[:64 << 20], 5)
    assert 3000.0 < st16 < 12000.0 and 3000.0 < tma < 12000.0, (st16, tma)
    assert pull > tma and pull < 60000.0, pull
    assert 0.5 < P.probe(P.PROBE_LAUNCH_PDL, None, 200) < 50.0
    assert 0.5 < P.probe(P.PROBE_LAUNCH, None, 200) < 50.0
    with pytest.raises(ptq.PtqError) as e:
        P.probe(P.PROBE_TMA_STORE, buf[:1024], 5)
    assert e.value.status == 2
    with pytest.raises(ptq.PtqError) as e:
        P.probe(P.PROBE_STORE16, buf[64:], 5)                       # not 256-byte aligned
    assert e.value.status == 4
    torch.cuda.synchronize()
