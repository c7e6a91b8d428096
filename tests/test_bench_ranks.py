"""The benchmark's multi-rank arithmetic on CPU: two gloo ranks, no GPU.

With N > 1 the ranks run independent replicas (the optimizer step has no cross-GPU exchange); the
reported value is all ranks' steps over the slowest rank's time, and only rank 0 of the oracle arm
prints a line.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, value = bench.whole_job_value(10.0 * (rank + 1), steps=5, dist=dist)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = (ms, value)


def test_value_is_all_ranks_steps_over_the_slowest_rank():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29513, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        ms, value = res[rank]
        assert ms == 20.0                       # the slower rank's time, on every rank
        assert abs(value - world * 5 / 20e-3) < 1e-9


def test_single_process_value():
    sys.path.insert(0, ROOT)
    import bench
    ms, value = bench.whole_job_value(4.0, steps=8)
    assert ms == 4.0 and abs(value - 2000.0) < 1e-9


def test_reference_arm_prints_on_rank_0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
