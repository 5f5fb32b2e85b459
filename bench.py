#!/usr/bin/env python
"""Benchmark of the PTS W8A8 linear path (quantize + integer GEMM + dequantize) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

One step = one forward pass of every linear layer of the workload configuration over one batch of
seeded synthetic activations, through the C ABI (`ptq_linear_forward`).  Prints ONE JSON line.

  value          INT8 TOPS = sum_layers 2 M K N / step time, inputs resident in HBM, CUDA events
  e2e            the same metric with pinned HOST buffers: host->device copy of x, forward,
                 device->host copy of y, every step, all inside the timed region (the three stages
                 run on three streams, double buffered, so copies and kernels overlap)
  roofline       the dominant kernel (largest share of the step), timed alone with CUDA events on
                 the launching stream in the same process; plus `kernels` with every kernel's figure
  cpu_baseline   the CPU oracle, as it stands, on a bounded row sample of the same workload

With N > 1 (torchrun) every rank runs an independent replica on its own GPU (the path has no
exchange step: rows are independent and the parameters are replicated), so scaling is weak.
`--impl reference` times the CPU oracle instead (rank 0 only).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "PTS W8A8 linear INT8 TOPS (quant+GEMM+dequant)"
UNIT = "TOPS"
INT8_OVER_BF16 = 2.0          # nominal dense ratio 4.5 / 2.25 PFLOP/s
INT8_NOMINAL_TOPS = 4500.0    # dense INT8 peak of one B200 (vendor datasheet)
SUSTAIN_SECONDS = 1.0         # length of the sustained leg; also the region length from which the sustained peak applies
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def layer_ops(spec, B):
    return 2.0 * B * spec.T * spec.K * spec.N


def workload_specs(name):
    from paper_2412_20386_b200 import workloads as wl
    idx = int(name[1:])
    return wl.configs()[idx]


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1, s0, s1):
        """Two summaries: the samples taken in [t0, t1] (the headline region) and in [s0, s1] (the
        sustained leg).  A headline region too short to hold three samples takes the sustained leg's
        clocks (same kernels, longer run) and says so in `window`."""
        empty = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return dict(empty), dict(empty)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()

        def summary(a, b):
            sm, smax, reasons = [], [], set()
            names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
            for ts, line in self.lines:
                if not (a <= ts <= b):
                    continue
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 6:
                    continue
                try:
                    sm.append(float(parts[0]))
                    smax.append(float(parts[1]))
                except ValueError:
                    continue
                for n, v in zip(names, parts[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                    "reasons": sorted(reasons), "samples": len(sm)}

        head, sus = summary(t0, t1), summary(s0, s1)
        head["window"] = "timed region"
        if head["samples"] < 3:
            head = dict(sus)
            head["window"] = "sustained leg (the timed region is shorter than three 50 ms samples)"
        return head, sus


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (also the cpu_baseline leg of the GPU arm)
# ------------------------------------------------------------------------------------------------
def oracle_layer_inputs(spec, rows):
    """Inputs of one layer restricted to the first `rows` token rows (whole images)."""
    import oracle
    from paper_2412_20386_b200 import workloads as wl
    images = max(1, min(spec.B, (rows + spec.T - 1) // spec.T))
    x = wl.activations(spec, wl.ROLE_EVAL, B=images).reshape(-1, spec.K)
    wq, dw, bias = wl.weights(spec)
    s, dx = oracle.calibrate(wl.activations(spec, wl.ROLE_CALIB), wq, dw)
    return x, wq, dw, bias, s, dx


def plan_oracle(specs, target_seconds):
    """Sizes a row sample per layer (leading rows, whole images generated) so that one pass of the
    oracle over all layers takes about `target_seconds`; a short probe per layer gives its rate."""
    import oracle
    total_ops_full = sum(layer_ops(sp, sp.B) for sp in specs)
    data = []
    for sp in specs:
        probe_rows = min(sp.M, 128)
        x, wq, dw, bias, s, dx = oracle_layer_inputs(sp, probe_rows)
        t0 = time.perf_counter()
        oracle.linear_forward(x, sp.T, wq, dw, s, dx, bias, rows=(0, probe_rows))
        dt = max(time.perf_counter() - t0, 1e-6)
        share = layer_ops(sp, sp.B) / total_ops_full
        rows = int(min(sp.M, max(8, probe_rows * (target_seconds * share) / dt)))
        if rows > x.shape[0]:
            x, wq, dw, bias, s, dx = oracle_layer_inputs(sp, rows)
        data.append((sp, rows, (x, wq, dw, bias, s, dx)))
    sample = "; ".join("c%d L%d %s: first %d of %d rows" % (sp.config, sp.layer, sp.name, rows, sp.M)
                       for sp, rows, _ in data[:6])
    if len(data) > 6:
        sample += "; ... (%d layers)" % len(data)
    return data, sample


def run_oracle_pass(data):
    """One pass of the oracle's whole path over the planned samples: (ops, seconds)."""
    import oracle
    ops = 0.0
    secs = 0.0
    for sp, rows, (x, wq, dw, bias, s, dx) in data:
        t0 = time.perf_counter()
        oracle.linear_forward(x, sp.T, wq, dw, s, dx, bias, rows=(0, rows))
        secs += time.perf_counter() - t0
        ops += 2.0 * rows * sp.K * sp.N
    return ops, secs


def time_oracle(specs, target_seconds):
    """(TOPS, sample text, seconds, per-phase seconds) of one oracle pass sized to about `target_seconds`.
    The phases (quantize, integer matmul, dequantize) are timed in a second pass over the same sample."""
    import oracle
    data, sample = plan_oracle(specs, target_seconds)
    ops, secs = run_oracle_pass(data)
    phases = {"quantize": 0.0, "int_matmul": 0.0, "dequant": 0.0}
    for sp, rows, (x, wq, dw, bias, s, dx) in data:
        xr = x[:rows]
        t0 = time.perf_counter()
        q = oracle.quantize(xr, sp.T, s, dx)
        t1 = time.perf_counter()
        acc = oracle.int_matmul(q, wq)
        t2 = time.perf_counter()
        oracle.dequant(acc, sp.T, dx, dw, bias)
        t3 = time.perf_counter()
        phases["quantize"] += t1 - t0
        phases["int_matmul"] += t2 - t1
        phases["dequant"] += t3 - t2
    return ops / secs / 1e12, sample, secs, {k: round(v, 4) for k, v in phases.items()}


def run_reference(args, specs, rank):
    """The reference arm: the CPU oracle, as it stands, on the host cores.  Each step is one pass over
    a bounded row sample of the workload, sized so that warm-up plus steps stay within ~2.5 minutes."""
    if rank != 0:
        return
    import oracle
    per_step = min(2.0, max(0.01, 150.0 / max(1, args.steps + args.warmup)))
    data, sample = plan_oracle(specs, per_step)
    for _ in range(args.warmup):
        run_oracle_pass(data)
    ops = secs = 0.0
    for _ in range(args.steps):
        o, t = run_oracle_pass(data)
        ops += o
        secs += t
    value = ops / secs / 1e12
    cores = oracle.num_threads()
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "n_layers": len(specs), "path": "cpu oracle"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def reduce_max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks of the default process group (the job's
    time is the slowest rank's); the identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def pct_of_peak(tops_per_gpu, region_seconds, int8_burst, int8_sustained):
    """Per-GPU throughput as a percentage of the nominal dense INT8 peak and of the measured proxy that
    fits the length of the timed region: 2 x bf16 burst below SUSTAIN_SECONDS, 2 x bf16 sustained from there."""
    long_run = region_seconds >= SUSTAIN_SECONDS
    proxy = int8_sustained if long_run else int8_burst
    return {"nominal_4500": 100.0 * tops_per_gpu / INT8_NOMINAL_TOPS,
            "measured_proxy": 100.0 * tops_per_gpu / proxy,
            "proxy": "2 x bf16_tflops%s = %.0f TOPS (timed region %.3f s)" % ("_sustained" if long_run else "", proxy,
                                                                             region_seconds)}


def whole_job_tops(world, step_ops_per_rank, ms_per_step):
    """Replicas: every rank does step_ops_per_rank in the (max over ranks) step time."""
    return world * step_ops_per_rank / (ms_per_step * 1e-3) / 1e12


def event_times_ms(torch, fn, iters):
    """Average device time of fn() per call, each call bracketed by its own CUDA events on the
    current stream (the stream the library launches on)."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    torch.cuda.synchronize()
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    ts = [a.elapsed_time(b) for a, b in evs]
    return sum(ts) / len(ts), min(ts), statistics.median(ts)


def region_time_ms(torch, fn, iters, warm=3):
    """Average device time per call of fn() over `iters` calls launched back to back between ONE pair of
    CUDA events on the current stream: the kernel's launch duration as it occurs inside a step, where the
    next launch's set-up overlaps the tail of this one.  (event_times_ms brackets every call with its own
    events and so also counts the launch gap of a kernel run in isolation.)"""
    for _ in range(warm):
        fn()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(iters):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / iters


def run_ours(args, specs, rank, world, local_rank):
    import torch
    import __graft_entry__ as entry
    if rank == 0:
        entry.build()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    import paper_2412_20386_b200 as ptq
    from paper_2412_20386_b200 import workloads as wl
    L = ptq.load_library()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks, peaks_kind = load_peaks()

    flags = {"unfused": 0, "fused": ptq.FLAG_FUSED_PROLOGUE, "pair": ptq.FLAG_CTA_PAIR}[args.path]
    layers = []
    for sp in specs:
        x_host = torch.from_numpy(wl.activations(sp, wl.ROLE_EVAL)).pin_memory()
        wq, dw, bias = wl.weights(sp)
        xcal = torch.from_numpy(wl.activations(sp, wl.ROLE_CALIB)).to(dev)
        if args.scheme == "w4a4":
            # 4-bit stand-ins for the workload's weights, packed two per byte (low nibble = even column)
            w4 = np.clip(np.rint(wq.astype(np.float32) / 18.0), -8, 7).astype(np.int32)
            if w4.shape[1] % 2:
                w4 = np.concatenate([w4, np.zeros((w4.shape[0], 1), np.int32)], axis=1)
            packed = (((w4[:, 1::2] << 4) | (w4[:, 0::2] & 15)) & 0xff).astype(np.uint8)
            s, dx = ptq.calibrate_w4a4(xcal, packed, sp.K, dw)
            layer = ptq.PtqLinear(packed, dw, s, dx, bias, packed4_K=sp.K)
        elif args.scheme == "pts-asym":
            s, dx, z = ptq.calibrate_asym(xcal, wq, dw)          # Q0 on the GPU, with zero offsets
            layer = ptq.PtqLinear(wq, dw, s, dx, bias, act_zero=z)
        else:
            # Q0 on the GPU; `static` is the per-tensor comparator: one step for all token positions
            s, dx = ptq.calibrate(xcal, wq, dw, per_tensor=(args.scheme == "static"))
            layer = ptq.PtqLinear(wq, dw, s, dx, bias)
        x_dev = x_host.to(dev)
        y_dev = torch.empty((sp.B, sp.T, sp.N), dtype=torch.float16, device=dev)
        y_host = torch.empty((sp.B, sp.T, sp.N), dtype=torch.float16).pin_memory()
        ws_bytes = layer.workspace_bytes_dynamic(sp.B) if args.scheme == "dynamic" else layer.workspace_bytes(sp.B, flags)
        ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
        layers.append(dict(spec=sp, layer=layer, x_host=x_host, x=x_dev, y=y_dev, y_host=y_host, ws=ws,
                           fused=bool((flags & ptq.FLAG_FUSED_PROLOGUE) and layer.fused_supported())))
    step_ops = sum(layer_ops(d["spec"], d["spec"].B) for d in layers)
    touched = sum(d["x"].numel() * 2 + d["y"].numel() * 2 for d in layers)

    def forward(d, x=None, y=None):
        x = d["x"] if x is None else x
        y = d["y"] if y is None else y
        if args.scheme == "dynamic":
            d["layer"].forward_dynamic(x, y=y, workspace=d["ws"])
        else:
            d["layer"].forward(x, y=y, workspace=d["ws"], flags=flags)

    def step():
        for d in layers:
            forward(d)

    # End to end: every step copies every layer's x from pinned host memory and every y back to it.
    # The three stages run on three streams with two device buffers per tensor, so the copy-in of the
    # next item, the kernels of this one and the copy-out of the previous one overlap (PCIe is full
    # duplex); events order each buffer's reuse.
    comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    for d in layers:
        d["xb"] = [d["x"], torch.empty_like(d["x"])]
        d["yb"] = [d["y"], torch.empty_like(d["y"])]
        d["ev_in"] = [torch.cuda.Event(), torch.cuda.Event()]
        d["ev_comp"] = [torch.cuda.Event(), torch.cuda.Event()]
        d["ev_out"] = [torch.cuda.Event(), torch.cuda.Event()]
        d["n"] = 0

    def step_e2e():
        for d in layers:
            j, first = d["n"] & 1, d["n"] < 2
            d["n"] += 1
            with torch.cuda.stream(s_in):
                if not first:
                    s_in.wait_event(d["ev_comp"][j])          # the forward that last read this x buffer
                d["xb"][j].copy_(d["x_host"], non_blocking=True)
                d["ev_in"][j].record(s_in)
            comp.wait_event(d["ev_in"][j])
            if not first:
                comp.wait_event(d["ev_out"][j])               # the copy-out that last read this y buffer
            forward(d, d["xb"][j], d["yb"][j])
            d["ev_comp"][j].record(comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(d["ev_comp"][j])
                d["y_host"].copy_(d["yb"][j], non_blocking=True)
                d["ev_out"][j].record(s_out)

    def drain_e2e():
        comp.wait_stream(s_in)
        comp.wait_stream(s_out)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- optional CUDA graph: one capture of the whole step, replayed (for launch-bound workloads) ---
    launches_per_step = None
    if args.graph:
        step()                                   # first calls outside the capture (one-time set-up in the library)
        torch.cuda.synchronize()
        n_before = ptq.binding.kernel_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        launches_per_step = ptq.binding.kernel_launch_count() - n_before
        eager_step = step
        step = graph.replay

    # ---- device-resident timing -------------------------------------------------------------
    # (1) the headline: exactly `steps` steps between one event pair; (2) the same steps again, each with
    # its own event pair (median and minimum, the protocol of the paper's Appendix B.2); (3) a sustained
    # leg: the step repeated for at least SUSTAIN_SECONDS, long enough for the clock samples (every
    # 50 ms) to fall inside it and for the power cap to act, reported beside the headline.
    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    n0 = ptq.binding.kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_start = time.time()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    t_end = time.time()
    launches = ptq.binding.kernel_launch_count() - n0
    if launches_per_step is not None:
        launches = launches_per_step * args.steps     # replayed from the captured graph
    ms_total = e0.elapsed_time(e1)
    for d in layers:
        d["layer"].device_status()

    n_each = max(3, min(args.steps, 200))
    _, step_min, step_med = event_times_ms(torch, step, n_each)

    n_sus = int(min(200000, max(args.steps, args.sustain_seconds * 1e3 / max(ms_total / args.steps, 1e-4))))
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ts0 = time.time()
    g0.record()
    for _ in range(n_sus):
        step()
    g1.record()
    barrier()
    ts1 = time.time()
    ms_sus = g0.elapsed_time(g1) / n_sus

    # ---- end to end with host buffers -------------------------------------------------------
    for _ in range(min(args.warmup, 3)):
        step_e2e()
    drain_e2e()
    barrier()
    e2e_steps = max(3, min(args.steps, 20))
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(e2e_steps):
        step_e2e()
    drain_e2e()                                   # the last copy-out is inside the timed region
    f1.record()
    barrier()
    ms_e2e = f0.elapsed_time(f1) / e2e_steps
    clocks, clocks_sus = sampler.stop(t_start, t_end, ts0, ts1)

    ms_total, ms_e2e, ms_sus = reduce_max_over_ranks([ms_total, ms_e2e, ms_sus], dev)
    ms_step = ms_total / args.steps
    value = whole_job_tops(world, step_ops, ms_step)
    e2e_value = whole_job_tops(world, step_ops, ms_e2e)

    if rank != 0:
        return

    # ---- per-kernel timing (rank 0): each kernel alone, events around every launch ----------
    # Kernels timed alone (50 launches, a few milliseconds, full clock) are rated against the BURST proxy
    # 2 x bf16_tflops; the sustained proxy applies only to regions of a second or more.
    int8_burst = peaks["bf16_tflops"] * INT8_OVER_BF16
    int8_sustained = peaks["bf16_tflops_sustained"] * INT8_OVER_BF16
    int8_peak = int8_burst
    hbm_peak = peaks["hbm_gbs"]
    kernels = []
    iters = 50
    for d in layers:
        sp, layer = d["spec"], d["layer"]
        M, K, N = sp.M, sp.K, sp.N
        tag = "c%d.L%d.%s" % (sp.config, sp.layer, sp.name)
        if d["fused"]:
            fwd = lambda: layer.forward(d["x"], y=d["y"], workspace=d["ws"], flags=flags)
            _, mn, med = event_times_ms(torch, fwd, iters)
            avg = region_time_ms(torch, fwd, iters)
            byts = 2.0 * M * K + N * K + 2.0 * M * N
            kernels.append(dict(kernel="ptq_fused_linear_kernel", layer=tag, ms=avg, ms_single_median=med, ms_single_min=mn,
                                ops=2.0 * M * K * N, bytes=byts))
        elif args.scheme == "dynamic":
            # the row-step quantizer has no entry point of its own: forward minus the GEMM timed alone
            pitch = layer.code_pitch()
            forward(d)
            tot = region_time_ms(torch, lambda: forward(d), iters)
            g_avg = region_time_ms(torch, lambda: layer.gemm_dequant(d["ws"][:M * pitch], sp.B, y=d["y"]), iters)
            q_ms = max(tot - g_avg, 1e-6)
            kernels.append(dict(kernel="ptq_quantize_dynamic_kernel", layer=tag, ms=q_ms, ops=0.0,
                                bytes=3.0 * M * K + 4.0 * M))
            kernels.append(dict(kernel="ptq_gemm_dequant_kernel", layer=tag, ms=g_avg, ops=2.0 * M * K * N,
                                bytes=1.0 * M * K + N * K + 2.0 * M * N))
        else:
            pitch = layer.code_pitch()
            codes = d["ws"][:M * pitch]
            qdense = torch.empty((sp.B, sp.T, K), dtype=torch.int8, device=dev)
            # cold: four input copies in rotation (more than L2 between two uses of one); warm: one buffer
            n_rot = 4 if 4 * d["x"].numel() * 2 <= 2e9 else 1
            x_rot = [d["x"]] + [d["x"].clone() for _ in range(n_rot - 1)]
            turn = [0]

            def quantize_rotating():
                turn[0] = (turn[0] + 1) % n_rot
                layer.quantize(x_rot[turn[0]], q=qdense)
            _, mn, med = event_times_ms(torch, quantize_rotating, iters)
            avg = region_time_ms(torch, quantize_rotating, iters)
            warm = region_time_ms(torch, lambda: layer.quantize(d["x"], q=qdense), iters)
            torch.cuda.synchronize()
            lo_code, hi_code = (0, 255) if args.scheme == "pts-asym" else ((-8, 7) if args.scheme == "w4a4" else (-128, 127))
            qv = qdense.view(torch.uint8) if args.scheme == "pts-asym" else qdense
            clip = float(((qv == lo_code) | (qv == hi_code)).float().mean().item())
            del x_rot
            kernels.append(dict(kernel="ptq_quantize_kernel", layer=tag, ms=avg, ms_single_median=med, ms_single_min=mn,
                                ms_l2_warm=warm, ops=0.0, bytes=3.0 * M * K, clip_rate=clip))
            layer.forward(d["x"], y=d["y"], workspace=d["ws"], flags=0)      # leaves valid codes in ws
            if flags & ptq.FLAG_CTA_PAIR:                                    # time the pair GEMM as forward minus quantize
                tot = region_time_ms(torch, lambda: layer.forward(d["x"], y=d["y"], workspace=d["ws"], flags=flags), iters)
                avg = mn = med = max(tot - avg, 1e-6)
            else:
                gemm = lambda: layer.gemm_dequant(codes, sp.B, y=d["y"])
                _, mn, med = event_times_ms(torch, gemm, iters)
                avg = region_time_ms(torch, gemm, iters)
            gname = ("ptq_gemm_dequant_pair_kernel" if flags & ptq.FLAG_CTA_PAIR else
                     ("ptq_gemm_dequant_kernel", "ptq_gemm_dequant_kernel<teams>", "ptq_gemm_dequant_panel_kernel")[layer.gemm_variant(sp.B)])
            kernels.append(dict(kernel=gname, layer=tag, ms=avg, ms_single_median=med, ms_single_min=mn,
                                ops=2.0 * M * K * N, bytes=1.0 * M * K + N * K + 2.0 * M * N))
            del qdense
    for k in kernels:
        t = k["ms"] * 1e-3
        k["tops"] = k["ops"] / t / 1e12
        k["gbs"] = k["bytes"] / t / 1e9
        k["frac_tensor"] = k["tops"] / int8_peak
        k["frac_tensor_nominal"] = k["tops"] / INT8_NOMINAL_TOPS
        k["frac_hbm"] = k["gbs"] / hbm_peak
        k["bound"] = "tensor" if k["frac_tensor"] >= k["frac_hbm"] else "hbm"
    # the dominant kernel is the one with the largest share of the step when timed alone
    family = lambda name: "gemm" if name.startswith("ptq_gemm_dequant") else name   # the GEMM variants count as one kernel
    agg = {}
    for k in kernels:
        agg.setdefault(family(k["kernel"]), 0.0)
        agg[family(k["kernel"])] += k["ms"]
    dom_name = max(agg, key=agg.get)
    dom = max((k for k in kernels if family(k["kernel"]) == dom_name), key=lambda k: k["ms"])
    if dom["bound"] == "tensor":
        roof = {"bound": "tensor", "achieved": dom["tops"], "peak": int8_peak, "unit": "TFLOP/s",
                "frac": dom["frac_tensor"], "frac_of_nominal_4500": dom["frac_tensor_nominal"]}
    else:
        roof = {"bound": "hbm", "achieved": dom["gbs"], "peak": hbm_peak, "unit": "GB/s", "frac": dom["frac_hbm"]}
    roof.update({"kernel": dom["kernel"], "layer": dom["layer"], "ms_per_launch": dom["ms"],
                 "peak_source": "%s (%s)" % (("2 x bf16_tflops, the burst figure: the kernel is timed alone, %d launches back "
                                              "to back between one pair of CUDA events" % iters
                                              if dom["bound"] == "tensor" else "hbm_gbs"), peaks_kind),
                 "traffic": TRAFFIC.get((dom["kernel"], args.workload, dom["layer"].split(".")[-1]))
                 if args.scheme == "pts" else None})

    # ---- what this GPU does for the bare data movements of the GEMM kernel (library probes, nothing else running)
    scratch = torch.empty(448 << 20, dtype=torch.uint8, device=dev)
    rates = {"store16_gbs": ptq.binding.probe(ptq.binding.PROBE_STORE16, scratch, 10),
             "tma_store_epilogue_pattern_gbs": ptq.binding.probe(ptq.binding.PROBE_TMA_STORE, scratch, 10),
             "operand_pull_l2_to_sm_gbs": ptq.binding.probe(ptq.binding.PROBE_OPERAND_PULL, scratch[:64 << 20], 10),
             "empty_launch_us": ptq.binding.probe(ptq.binding.PROBE_LAUNCH, None, 500),
             "empty_launch_pdl_us": ptq.binding.probe(ptq.binding.PROBE_LAUNCH_PDL, None, 500)}
    rates = {k: round(v, 2) for k, v in rates.items()}
    del scratch

    # ---- CPU oracle baseline on a bounded sample -------------------------------------------
    import oracle
    cpu_val, cpu_sample, cpu_secs, cpu_phases = time_oracle(specs, args.cpu_seconds)
    cpu = {"value": cpu_val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": cpu_sample, "seconds": cpu_secs, "phase_seconds": cpu_phases}

    h2d = sum(d["x"].numel() * 2 for d in layers)
    d2h = sum(d["y"].numel() * 2 for d in layers)
    sp0 = specs[0]
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "layers": ["%s %dx%d->%d" % (sp.name, sp.M, sp.K, sp.N) for sp in specs][:8],
                   "n_layers": len(specs), "batch": sp0.B, "tokens": sp0.T, "path": args.path,
                   "cuda_graph": bool(args.graph), "scheme": args.scheme,
                   "fused_layers": sum(1 for d in layers if d["fused"]),
                   "l2": "inputs_larger_than_l2 (%.0f MB touched per step)" % (touched / 1e6)
                   if touched > 2 * 126e6 else "working set %.0f MB fits L2: L2-warm timing" % (touched / 1e6),
                   "parallelism": "replicas x%d" % world},
        "ms_per_step_median": step_med, "ms_per_step_min": step_min,
        "pct_of_int8_peak": pct_of_peak(value / world, ms_total * 1e-3, int8_burst, int8_sustained),
        "clocks": clocks,
        "sustained": {"seconds": round(ms_sus * n_sus * 1e-3, 3), "steps": n_sus, "ms_per_step": ms_sus,
                      "value": whole_job_tops(world, step_ops, ms_sus), "unit": UNIT,
                      "pct_of_int8_peak": pct_of_peak(whole_job_tops(1, step_ops, ms_sus), ms_sus * n_sus * 1e-3,
                                                      int8_burst, int8_sustained),
                      "clocks": clocks_sus,
                      "ms_x_mhz": (ms_sus * clocks_sus["sm_mhz"]) if clocks_sus.get("sm_mhz") else None,
                      "headline_ms_x_max_mhz": (ms_step * clocks_sus["sm_max_mhz"]) if clocks_sus.get("sm_max_mhz") else None},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e},
        "gpu_launches": int(launches),
        "roofline": roof,
        "measured_rates": rates,
        "kernels": [{k2: (round(v, 5) if isinstance(v, float) else v) for k2, v in k.items()} for k in kernels[:16]],
        "cpu_baseline": cpu,
    }
    print(json.dumps(out))


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised
# under profiles/; keyed by (kernel, workload, layer).  An entry is removed when its kernel changes.
TRAFFIC = {
    ("ptq_gemm_dequant_panel_kernel", "c3", "in_proj"): 41.190144e6 + 250.822144e6,
    ("ptq_gemm_dequant_kernel", "c3", "out_proj"): 78.705408e6 + 33.518592e6,
    ("ptq_quantize_kernel", "c3", "in_proj"): 77.492224e6 + 6.748672e6,
    ("ptq_quantize_kernel", "c3", "out_proj"): 155.017472e6 + 22.338304e6,
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c0", "c1", "c2", "c3", "c4"])
    ap.add_argument("--path", default="unfused", choices=["unfused", "fused", "pair"],
                    help="unfused: quantize kernel + GEMM kernel (fastest at present, the default); "
                         "fused: PTQ_FLAG_FUSED_PROLOGUE; pair: PTQ_FLAG_CTA_PAIR")
    ap.add_argument("--scheme", default="pts", choices=["pts", "static", "pts-asym", "dynamic", "w4a4"],
                    help="pts: symmetric per-token-static codes (the default); static: the per-tensor static comparator "
                         "(one step for the whole tensor, same kernels); pts-asym: with a zero offset per token "
                         "position; dynamic: the per-token dynamic comparator (row steps measured at run time); "
                         "w4a4: 4-bit codes and packed 4-bit weights on the 8-bit tensor-core path")
    ap.add_argument("--graph", action="store_true",
                    help="capture one step in a CUDA graph and time replays (for launch-bound workloads such as c1)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--sustain-seconds", type=float, default=SUSTAIN_SECONDS,
                    help="length of the sustained leg that follows the timed region (profiling runs shorten it)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    specs = workload_specs(args.workload)

    if args.impl == "reference":
        run_reference(args, specs, rank)
        return

    if world > 1:
        import torch
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl")
    try:
        run_ours(args, specs, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
