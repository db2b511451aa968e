"""The benchmark's multi-rank bookkeeping (replicas only: no data-path collective) on CPU with gloo, world size 2."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                 # rank 1 is the slow one
        dist.barrier()
        worst = bench.max_over_ranks(local_ms, world, "cpu")
        out[rank] = (worst, bench.job_value(8.0 * 64 ** 3, world, worst))
    finally:
        dist.destroy_process_group()


def test_step_time_is_max_over_ranks_and_value_is_whole_job():
    world = 2
    port = 29500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1]
    worst, value = out[0]
    assert worst == 15.0
    assert value == pytest.approx(2 * 8.0 * 64 ** 3 / 15.0e-3 / 1e12)


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.job_value(1e12, 1, 1000.0) == pytest.approx(1.0)
