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
