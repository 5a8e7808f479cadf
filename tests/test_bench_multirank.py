"""The N > 1 path of bench.py on CPU: ranks are independent replicas (no data-path collective), the job's
time is the slowest rank's, the value is the sum of what all replicas moved over that time; and under a
multi-rank launch only rank 0 of the reference arm works and prints.  world_size 2, gloo."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = [10.0, 12.5][rank]                                   # rank 1 is the slower replica
    agreed = bench.max_over_ranks(ms, dist, torch.device("cpu"))
    q.put((rank, agreed, bench.replica_throughput(world, 4.0e9, agreed)))
    dist.barrier()
    dist.destroy_process_group()


def test_replicas_time_is_the_slowest_rank_and_value_is_the_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, agreed, value in got:
        assert agreed == 12.5                                 # max over ranks, the same on every rank
        assert value == pytest.approx(2 * 4.0e9 / 12.5e-3 / 1e9)


def test_single_process_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.25, None, torch.device("cpu")) == 3.25
    assert bench.replica_throughput(1, 1.0e9, 1.0) == pytest.approx(1000.0)


def test_reference_arm_only_rank0_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""      # the other ranks exit 0 without work
