"""Batch-sharded filtered backward over a process group.

Every step of the method is per image except the sum over the batch in Eq. (grad_w), which is
linear: rank k runs the path on its own images (stash, gradient filter, g_X -- no exchange) and
gets a partial g_W; one all-reduce (sum) of g_W finishes the layer.  For r >= 2 every tap of an
input/output channel pair carries the same value, so only the unique-value matrix
[C_out, C_in/groups] crosses the wire and is written back to all taps.  torch.distributed is the
plumbing (NCCL between GPUs, gloo in the CPU tests of this host logic); the arithmetic of the path
stays in the CUDA library.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(N: int, rank: int, world: int) -> tuple[int, int]:
    """Images [lo, hi) of rank `rank`: contiguous, sizes differing by at most one."""
    base, extra = divmod(N, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def all_reduce_weight_gradient(g_W: torch.Tensor, r: int, group=None) -> torch.Tensor:
    """Sums the ranks' partial g_W [C_out, C_ig, KH, KW] in place and returns it."""
    if r >= 2 and g_W.shape[2] * g_W.shape[3] > 1:
        uniq = g_W[:, :, 0, 0].contiguous()              # all taps are equal: reduce one of them
        dist.all_reduce(uniq, op=dist.ReduceOp.SUM, group=group)
        g_W.copy_(uniq[:, :, None, None].expand_as(g_W))
    else:
        dist.all_reduce(g_W, op=dist.ReduceOp.SUM, group=group)
    return g_W


def sharded_backward(gf, desc_local, g_y, stash, W, g_W, g_X, workspace, group=None, stream=None) -> None:
    """gf_backward on this rank's images (desc_local.N = its share of the batch), then the
    all-reduce of g_W.  g_X is this rank's part of the input gradient and is complete as it is."""
    gf.gf_backward(desc_local, g_y, stash, W, g_W, g_X, workspace, None, stream)
    if g_W is not None:
        if stream is not None and isinstance(stream, torch.cuda.Stream):
            with torch.cuda.stream(stream):
                all_reduce_weight_gradient(g_W, desc_local.r, group)
        else:
            all_reduce_weight_gradient(g_W, desc_local.r, group)
