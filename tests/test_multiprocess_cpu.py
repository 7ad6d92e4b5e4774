"""Host logic of the multi-GPU benchmark path (replicas only: a barrier and a
max over ranks, no data-path collective), run as two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch
import bench
rank, local, world = bench._dist_setup(2, backend="gloo")
assert world == 2 and rank == int(os.environ["RANK"])
bench._barrier(world)
ms = bench._barrier_max(world, 10.0 + 5.0 * rank, torch.device("cpu"))    # rank 1 is the slow one
bench._barrier(world)
print(json.dumps({"rank": rank, "ms": ms, "value": bench.aggregate_value(world, 30, ms)}))
import torch.distributed as dist
dist.destroy_process_group()
"""


def test_two_ranks_agree_on_the_slowest_time():
    port = 29500 + os.getpid() % 2000
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    assert {o["rank"] for o in outs} == {0, 1}
    for o in outs:
        assert o["ms"] == 15.0                      # max over ranks
        assert abs(o["value"] - 2 * 30 / 0.015) < 1e-6     # whole-job iterations per second


def test_reference_arm_only_rank_zero_prints():
    """Under a multi-rank launch the CPU-oracle arm runs on rank 0 alone."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg1",
                        "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
