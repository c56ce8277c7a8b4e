"""The N > 1 path on CPU (gloo, world size 2).  The hot path has no exchange step, so ranks run independent
replicas; what is multi-rank is the timing reduction (slowest rank), the aggregate value, and who prints."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 * (rank + 1), dist, "cpu")          # rank 1 is the slow one
val = bench.aggregate_value(15, 4, ms, world)
dist.barrier()
if rank == 0:
    print(json.dumps(dict(ms=ms, value=val, world=world)))
dist.destroy_process_group()
'''


def _torchrun(args, timeout=300):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29613"] + args
    return subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, env=env, cwd=ROOT)


def test_slowest_rank_sets_the_time_and_value_is_the_aggregate(tmp_path):
    w = tmp_path / "worker.py"
    w.write_text(WORKER % ROOT)
    r = _torchrun([str(w)])
    assert r.returncode == 0, r.stderr[-2000:]
    line = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(line) == 1                                            # rank 0 alone prints
    d = json.loads(line[0])
    assert d["world"] == 2 and d["ms"] == 20.0                       # max over ranks
    assert d["value"] == pytest.approx(2 * 15 * 4 / 20e-3)           # both replicas' units over the slowest time


def test_reference_arm_under_torchrun_prints_once():
    r = _torchrun(["bench.py", "--impl", "reference", "--workload", "linear", "--gpus", "2", "--steps", "1",
                   "--warmup", "0"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0
