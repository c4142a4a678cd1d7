"""The multi-GPU form of the benchmark is "replicas": every rank runs the same per-GPU step on its own seeded
batch and only the elapsed time is reduced (max over ranks).  These CPU tests run that host logic with two
gloo ranks: rank-dependent seeds give different batches, the max-reduction picks the slowest rank, and the
reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import numpy as np, torch, torch.distributed as dist
from paper_1908_05858_b200 import synth
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
x, w = synth.conv_case(2, 2, 64, 8, 8, 64, 3, 3, salt=64 + 1000 * rank)   # the benchmark's per-rank recipe
digest = torch.tensor([float(np.abs(x).sum())], dtype=torch.float64)
all_d = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
dist.all_gather(all_d, digest)
t = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)   # pretend elapsed ms: rank 1 is slower
dist.barrier()
dist.all_reduce(t, op=dist.ReduceOp.MAX)
if rank == 0:
    print(json.dumps({"digests": [float(d.item()) for d in all_d], "max_ms": float(t.item()), "world": world}))
dist.destroy_process_group()
""" % ROOT


def run_torchrun(args, timeout=300):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", "29731"] + args
    return subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, env=env, cwd=ROOT)


def test_two_ranks_get_different_batches_and_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    r = run_torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["world"] == 2
    assert d["digests"][0] != d["digests"][1]   # different seeds per rank
    assert d["max_ms"] == 15.0                  # max over ranks, not rank 0's own time


def test_reference_arm_prints_once_under_two_ranks():
    r = run_torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "Gbit-ops/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
