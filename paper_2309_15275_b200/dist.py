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


class GwReducer:
    """Sums the g_W of several layers over the ranks while later layers still
    compute: the all-reduce of layer i is issued as soon as that layer's kernels
    are done, not after the whole batch call.

    On GPUs the reductions run on a stream of their own, each behind the event
    that lbp_backward_batch records for its layer (`events()` is what to pass as
    `done_events`); `reduce()` enqueues them and makes the current stream wait
    for the last one.  On CPU tensors (gloo) the reductions are started together
    as asynchronous operations and waited for in order.  The sums are the same as
    with one blocking all-reduce per layer after the call."""

    def __init__(self, n_layers: int, device=None):
        self.n = n_layers
        self.active = dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1
        self.cuda = self.active and device is not None and torch.device(device).type == "cuda"
        if self.cuda:
            self.stream = torch.cuda.Stream(device=device)
            self._events = [torch.cuda.Event() for _ in range(n_layers)]
            self._joined = torch.cuda.Event()
        else:
            self.stream, self._events, self._joined = None, None, None

    def events(self):
        """Events for lbp_backward_batch(done_events=...), or None when nothing is reduced."""
        return self._events

    def reduce(self, g_Ws):
        if not self.active:
            return g_Ws
        if len(g_Ws) != self.n:
            raise ValueError("one g_W per layer")
        if self.cuda:
            cur = torch.cuda.current_stream()
            with torch.cuda.stream(self.stream):
                for g, e in zip(g_Ws, self._events):
                    self.stream.wait_event(e)
                    dist.all_reduce(g, op=dist.ReduceOp.SUM)
                self._joined.record(self.stream)
            cur.wait_event(self._joined)          # the step ends when every g_W is summed
        else:
            handles = [dist.all_reduce(g, op=dist.ReduceOp.SUM, async_op=True) for g in g_Ws]
            for h in handles:
                h.wait()
        return g_Ws
