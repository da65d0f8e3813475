"""`torch.autograd` front end of the C ABI: a linear layer whose backward pass is
Algorithm 1 (low-rank backpropagation on the selected Walsh-Hadamard bases).

Only the backward pass is the library's: the forward product `y = x W^T` is a
plain matrix product and is left to torch.  The layer has no bias (the paper's
Eq. 1) and expects the token grid explicit: x of shape (B, H, W, Cin).
"""
from __future__ import annotations

from typing import Sequence, Tuple

import torch

from . import binding as _b


class LbpLinearFunction(torch.autograd.Function):
    """y = x W^T;  backward: (g_x, g_W) = lbp_backward(x, g_y, W, k, bases)."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, weight: torch.Tensor, k: int,
                bases: Sequence[Tuple[int, int]]):
        if x.dim() != 4:
            raise ValueError("x must be (B, H, W, Cin)")
        ctx.save_for_backward(x, weight)
        ctx.k, ctx.bases = int(k), [tuple(p) for p in bases]
        return torch.matmul(x, weight.t())

    @staticmethod
    def backward(ctx, g_y: torch.Tensor):
        x, weight = ctx.saved_tensors
        g_x, g_W = _b.lbp_backward(x.contiguous(), g_y.contiguous(), weight.contiguous(), ctx.k,
                                   ctx.bases, gw_dtype=weight.dtype)
        return g_x, g_W, None, None


class LbpLinear(torch.nn.Module):
    """Bias-free linear layer over a (B, H, W, C) token grid with LBP-WHT backward.

    `bases` is an ordered list of 0-based (i, j) sequency pairs, e.g. from
    `lbp_select_bases(k, SEL_L1, m)` (Eq. 8) or `lbp_select_lhe` (Sec. 3.2).
    """

    def __init__(self, in_features: int, out_features: int, k: int,
                 bases: Sequence[Tuple[int, int]], device=None, dtype=None):
        super().__init__()
        w = torch.empty((out_features, in_features), device=device, dtype=dtype)
        torch.nn.init.normal_(w, std=in_features ** -0.5)
        self.weight = torch.nn.Parameter(w)
        self.k, self.bases = int(k), [tuple(p) for p in bases]

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return LbpLinearFunction.apply(x, self.weight, self.k, self.bases)
