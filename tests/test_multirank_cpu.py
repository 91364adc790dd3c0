"""The N > 1 path of bench.py on CPU: two gloo ranks, replicas only (no data-path collective).  Each rank times its own
replica; the reported time is the maximum over ranks and the value is the whole-job aggregate."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_mine = 2.0 + rank                     # rank 1 is the slow replica
        ms = bench.max_over_ranks(ms_mine, dist, torch.device("cpu"))
        value = bench.whole_job_rate(1e12, world, ms)
        dist.barrier()
        out[rank] = (ms, value)
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate():
    world = 2
    port = 29500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert len(out) == world
    for rank in range(world):
        ms, value = out[rank]
        assert ms == pytest.approx(3.0)                      # max over ranks, identical everywhere
        assert value == pytest.approx(2 * 1e12 / 3e-3)       # two replicas' work over the slowest replica's time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.5, None, None) == 1.5
    assert bench.whole_job_rate(10.0, 1, 1000.0) == pytest.approx(10.0)
