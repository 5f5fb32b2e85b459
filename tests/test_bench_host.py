"""Host-side logic of bench.py that needs no GPU: the multi-rank reduction (world size 2 over gloo),
the whole-job aggregate, the reference arm's rank gating and the oracle sampling plan."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 is slower on the first, faster on the second
out = bench.reduce_max_over_ranks(ms)
dist.barrier()
print(json.dumps({"rank": rank, "world": world, "max": out,
                  "tops": bench.whole_job_tops(world, 2.0e12, out[0])}))
dist.destroy_process_group()
""" % ROOT


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_max_over_ranks_and_whole_job_value_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=180)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    for o in outs:
        assert o["world"] == 2
        assert o["max"] == [15.0, 3.0]                      # slowest rank per entry, same on every rank
        assert o["tops"] == pytest.approx(2 * 2.0e12 / 15e-3 / 1e12)


def test_single_process_reduction_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_tops(1, 1e12, 1.0) == pytest.approx(1000.0)


def test_reference_arm_runs_on_rank0_only_and_prints_the_contract_line():
    port = free_port()
    results = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--steps", "2", "--warmup", "1", "--workload", "c0"],
                           env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr
        results.append(r.stdout.strip())
    assert results[1] == ""                                   # other ranks exit 0 without work
    line = json.loads(results[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["steps"] == 2
    assert line["unit"] == "TOPS" and line["value"] > 0 and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"] == {"value": line["value"], "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_oracle_sampling_plan_is_bounded():
    sys.path.insert(0, ROOT)
    import bench
    specs = bench.workload_specs("c0")
    data, sample = bench.plan_oracle(specs, 0.05)
    assert len(data) == 1 and 8 <= data[0][1] <= specs[0].M and "rows" in sample
    ops, secs = bench.run_oracle_pass(data)
    assert ops == 2.0 * data[0][1] * specs[0].K * specs[0].N and secs > 0


def test_measured_proxy_follows_the_length_of_the_timed_region():
    sys.path.insert(0, ROOT)
    import bench
    short = bench.pct_of_peak(1500.0, 0.005, 3312.0, 2744.0)
    long_ = bench.pct_of_peak(1300.0, 1.2, 3312.0, 2744.0)
    assert short["nominal_4500"] == pytest.approx(100 * 1500 / 4500)
    assert short["measured_proxy"] == pytest.approx(100 * 1500 / 3312) and "sustained" not in short["proxy"]
    assert long_["measured_proxy"] == pytest.approx(100 * 1300 / 2744) and "bf16_tflops_sustained" in long_["proxy"]


def test_clock_summaries_keep_the_two_windows_apart():
    sys.path.insert(0, ROOT)
    import bench

    class FakeProc:
        def terminate(self):
            pass

        def wait(self, timeout=None):
            return 0

    smp = bench.ClockSampler(0)
    smp.proc = FakeProc()
    line = lambda mhz, cap: "%d, 1965, Not Active, Not Active, Not Active, %s" % (mhz, cap)
    smp.lines = [(10.00, line(1965, "Not Active")),                       # inside the 20 ms headline region
                 (11.0, line(1500, "Active")), (11.3, line(1400, "Active")), (11.6, line(1450, "Active")),
                 (30.0, line(300, "Not Active"))]                          # idle, outside both windows
    head, sus = smp.stop(9.99, 10.01, 10.9, 11.9)
    assert sus["sm_mhz"] == 1450 and sus["samples"] == 3 and sus["reasons"] == ["sw_power_cap"]
    assert head["samples"] == 3 and "sustained leg" in head["window"]     # one sample is too few: borrowed, and said so
    smp.proc = FakeProc()
    head, _ = smp.stop(10.9, 11.9, 10.9, 11.9)
    assert head["window"] == "timed region" and head["sm_max_mhz"] == 1965
