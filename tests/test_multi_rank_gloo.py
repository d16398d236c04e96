"""The N > 1 plumbing of bench.py, on CPU with the gloo backend (world size 2):
replicas draw different inputs, the timing is the maximum over ranks, the value
counts every replica's elements, only rank 0 reports, and the reference arm
leaves ranks > 0 idle."""

import json
import os
import subprocess
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, %(root)r)
import torch, torch.distributed as dist
import bench
from paper_2501_17392_b200 import workloads as W
rank, world, local = bench.dist_env()
dist.init_process_group("gloo", rank=rank, world_size=world)
w = W.scaled(W.WORKLOADS["cfg1"], 4096)
H = W.honest_updates(w, bench.replica_seed_round(rank), device="cpu")
mine_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
total_ms = bench.max_over_ranks(mine_ms, world, torch.device("cpu"))
sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
dist.all_gather(sums, H.double().sum().reshape(1))
dist.barrier()
if rank == 0:
    print(json.dumps({"total_ms": total_ms, "value": bench.whole_job_value(world, w.n, w.d, 5, total_ms),
                      "sums": [float(s) for s in sums], "n": w.n, "d": w.d}))
dist.destroy_process_group()
"""


def _env(rank, world, port):
    env = dict(os.environ)
    env.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1",
                "MASTER_PORT": str(port), "OMP_NUM_THREADS": "1"})
    return env


def test_two_ranks_max_time_and_whole_job_value(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % {"root": ROOT})
    port = 29500 + os.getpid() % 2000
    procs = [subprocess.Popen([sys.executable, str(script)], env=_env(r, 2, port), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (so, se) in zip(procs, outs):
        assert p.returncode == 0, se[-2000:]
    assert outs[1][0].strip() == ""                                   # only rank 0 reports
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["total_ms"] == 20.0                                   # the slowest rank sets the time
    assert line["value"] == 2 * line["n"] * line["d"] * 5 / 20e-3     # every replica's elements count
    assert line["sums"][0] != line["sums"][1]                         # replicas drew different inputs


def test_reference_arm_runs_on_rank_zero_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1", "--steps", "1",
           "--warmup", "1", "--gpus", "2"]
    r1 = subprocess.run(cmd, env=_env(1, 2, 29999), capture_output=True, text=True, timeout=240)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=_env(0, 2, 29999), capture_output=True, text=True, timeout=240)
    assert r0.returncode == 0, r0.stderr[-2000:]
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
    assert line["config"]["workload"] == "cfg1" and line["value"] > 0


def test_world_size_one_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.replica_seed_round(0) == 0 and bench.replica_seed_round(3) != bench.replica_seed_round(2)
