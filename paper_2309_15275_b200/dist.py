"""Data-parallel plumbing: one process per GPU, batch sharded by whole images.

k x k token blocks are independent, so x, g_y, x_hat, g_y_hat and g_x stay local
to the rank that owns the images.  The only exchange step of the path is the
sum of g_W over the batch (Algorithm 1 sums it over batch, blocks and bases):
one all-reduce of the (Cout, Cin) fp32 matrix, the same one plain data-parallel
backpropagation needs, independent of the rank r.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_images(B: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the images rank owns; shards differ by at most one image."""
    base, extra = divmod(B, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def allreduce_gw(g_W: torch.Tensor) -> torch.Tensor:
    """Sum g_W over all ranks in place (NCCL on GPUs, gloo on CPU); no-op for one rank."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(g_W, op=dist.ReduceOp.SUM)
    return g_W
