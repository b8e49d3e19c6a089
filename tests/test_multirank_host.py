"""Host logic of multi-rank bench runs (independent replicas, no collective on the data path), on CPU with gloo."""
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = [4.0, 6.5][rank]                          # rank 1 is the slow replica
        dist.barrier()
        ms = bench.max_over_ranks(local_ms, dist, "cpu")
        value = bench.job_throughput(64, world, ms * 1e-3)   # 64 tree rows per step and rank
        out[rank] = (ms, value)
    finally:
        dist.destroy_process_group()


def test_replica_timing_is_max_over_ranks_and_value_is_whole_job():
    world, port = 2, 29531 + os.getpid() % 200
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]                                  # every rank sees the same aggregate
    ms, value = res[0]
    assert ms == 6.5
    assert value == pytest.approx(2 * 64 / 6.5e-3)


def test_single_process_path_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25, None, "cpu") == 3.25
    assert bench.job_throughput(64, 1, 4e-3) == pytest.approx(16000.0)


def test_reference_arm_runs_on_rank_zero_only():
    """Under a multi-rank launch only rank 0 times the oracle; the other ranks exit 0 and print nothing."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "3", "--workload", "c1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    assert r.stdout.strip() == ""
