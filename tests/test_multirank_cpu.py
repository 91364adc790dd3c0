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


def test_gpus_flag_must_agree_with_the_launcher():
    """bench.py --gpus N under a launcher that started another number of ranks refuses to run (before touching a GPU)."""
    import subprocess
    env = dict(os.environ, WORLD_SIZE="4", RANK="0", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2"], env=env, capture_output=True, text=True)
    assert r.returncode != 0
    assert "4 ranks" in r.stderr


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself():
    """--gpus 2 with no launcher around: bench.py starts two ranks; on the reference arm (CPU only) rank 0 prints the one
    JSON line and the other rank exits 0 without work."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--cpu-rows", "2", "--cpu-features", "16"], env=env, capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0
