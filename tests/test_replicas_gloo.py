"""N > 1 is "replicas only": every rank runs the whole path on its own copy of the
workload and nothing crosses ranks but the timing reduction.  These tests run that
reduction on two CPU ranks over gloo, and the rank-0-only rule of the reference arm."""
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, times_ms, steps: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        ms = bench.max_over_ranks(times_ms[rank], dist, "cpu")
        out[rank] = (ms, bench.job_value_us(ms, steps, world))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_timing_is_max_over_ranks_and_value_counts_every_replica():
    world, steps = 2, 50
    times = [12.5, 20.0]                       # rank 1 is the slow replica
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), times, steps, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        ms, value = res[rank]
        assert ms == 20.0                       # every rank sees the slowest rank's time
        assert value == pytest.approx(20.0 * 1e3 / (steps * world))   # 100 layer steps in 20 ms


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.25, None, "cpu") == 3.25
    assert bench.job_value_us(10.0, 100, 1) == pytest.approx(100.0)


def test_reference_arm_runs_on_rank_0_only():
    """Under a multi-rank launch the CPU checker is timed by rank 0 alone; the other ranks
    exit 0 without output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0
    assert r.stdout.strip() == ""
