"""Batch sharding of a layer over a process group (paper_2301_00330_b200/sharded.py): the host
logic on two and three CPU ranks over gloo.  Every rank computes its shard's partial results with
the CPU oracle (this is a test: the product's arithmetic runs in the CUDA library), the wrapper's
all-reduce finishes Eq. (grad_w), and the result must equal the oracle on the whole batch."""
import os
import socket
import sys

import numpy as np
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


def _inputs(N=5, Cin=6, Cout=4, H=8, W=6, K=3):
    rng = np.random.default_rng(123)
    return (rng.normal(size=(N, Cin, H, W)), rng.normal(size=(N, Cout, H, W)), rng.normal(size=(Cout, Cin, K, K)))


def _worker(rank: int, world: int, port: int, r: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from paper_2301_00330_b200 import sharded
        x, gy, theta = _inputs()
        lo, hi = sharded.shard_range(x.shape[0], rank, world)
        stash = oracle.stash_forward(x[lo:hi], r)
        if hi > lo:
            gw, gx = oracle.backward(gy[lo:hi], stash, theta, r)
        else:                                   # a rank without images contributes zeros
            gw, gx = np.zeros_like(theta), np.zeros((0,) + x.shape[1:])
        g_W = torch.from_numpy(gw.copy())
        sharded.all_reduce_weight_gradient(g_W, r)
        out[rank] = (lo, hi, g_W.numpy(), gx)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,r", [(2, 2), (3, 2), (2, 1), (3, 4)])
def test_sharded_layer_equals_whole_batch(world, r):
    import oracle
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), r, out), nprocs=world, join=True)
        res = dict(out)
    x, gy, theta = _inputs()
    gw_ref, gx_ref = oracle.backward(gy, oracle.stash_forward(x, r), theta, r)
    covered = []
    for rank in range(world):
        lo, hi, gw, gx = res[rank]
        covered += list(range(lo, hi))
        assert np.allclose(gw, gw_ref, rtol=1e-12, atol=1e-12)          # every rank ends with the full g_W
        assert np.allclose(gx, gx_ref[lo:hi], rtol=1e-12, atol=1e-13)   # g_X needs no exchange
    assert covered == list(range(x.shape[0]))


def test_shard_ranges_partition_the_batch():
    from paper_2301_00330_b200 import sharded
    for N in (1, 5, 8, 128):
        for world in (1, 2, 3, 8):
            spans = [sharded.shard_range(N, k, world) for k in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == N
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
