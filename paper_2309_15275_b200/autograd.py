"""`torch.autograd` front end of the C ABI: a linear layer whose backward pass is
Algorithm 1 (low-rank backpropagation on the selected Walsh-Hadamard bases).

Only the backward pass is the library's: the forward product `y = x W^T` is a
plain matrix product and is left to torch.  The layer takes the token grid
explicit, x of shape (B, H, W, Cin), or, with `grid=(H, W)`, a token sequence
(B, n + H*W, Cin) whose first n tokens (class tokens) are not part of the grid:
those take exact backpropagation (Eq. 2), and the grid tokens are handed to the
library as a strided view of the sequence, without a copy.  The bias (absent
from the paper's Eq. 1) is optional.
"""
from __future__ import annotations

from typing import Sequence, Tuple

import torch

from . import binding as _b


class LbpLinearFunction(torch.autograd.Function):
    """y = x W^T (+ b);  backward: Algorithm 1 on the selected bases.

    With `save_projected` the forward pass keeps x_hat = p(x) (Eq. 3) instead of
    x: r / k^2 of the activation's elements stay alive until the backward pass,
    which then starts at the second step of Algorithm 1."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, weight: torch.Tensor, bias, k: int,
                bases: Sequence[Tuple[int, int]], save_projected: bool, grid=None):
        ctx.k, ctx.bases = int(k), [tuple(p) for p in bases]
        ctx.has_bias = bias is not None
        ctx.grid = None
        if grid is not None:
            H, W = int(grid[0]), int(grid[1])
            if x.dim() != 3 or x.shape[1] < H * W:
                raise ValueError("with a grid, x must be (B, n + H*W, Cin)")
            ctx.grid, ctx.projected = (H, W), False
            ctx.save_for_backward(x, weight)
            y = torch.matmul(x, weight.t())
            return y if bias is None else y + bias
        if x.dim() != 4:
            raise ValueError("x must be (B, H, W, Cin)")
        ctx.projected = bool(save_projected) and x.is_cuda
        if ctx.projected:
            ctx.save_for_backward(_b.lbp_project(x.contiguous(), ctx.k, ctx.bases), weight)
        else:
            ctx.save_for_backward(x, weight)
        y = torch.matmul(x, weight.t())
        return y if bias is None else y + bias

    @staticmethod
    def backward(ctx, g_y: torch.Tensor):
        saved, weight = ctx.saved_tensors
        g_b = (torch.empty(weight.shape[0], dtype=torch.float32, device=g_y.device)
               if ctx.has_bias else None)
        if ctx.grid is not None:
            return LbpLinearFunction._backward_sequence(ctx, saved, weight, g_y, g_b)
        g_y = g_y.contiguous()
        kw = {"x_hat": saved} if ctx.projected else {}
        g_x, g_W = _b.lbp_backward_ex(None if ctx.projected else saved.contiguous(), g_y,
                                      weight.contiguous(), ctx.k, ctx.bases, g_bias=g_b,
                                      gw_dtype=weight.dtype, **kw)
        return g_x, g_W, (None if g_b is None else g_b.to(weight.dtype)), None, None, None, None

    @staticmethod
    def _backward_sequence(ctx, x, weight, g_y, g_b):
        H, W = ctx.grid
        B, n_all, Cin = x.shape
        n = n_all - H * W
        x, g_y = x.contiguous(), g_y.contiguous()
        g_x = torch.empty_like(x)
        kw = {}
        if n > 0:
            # one class token per image: rows with the sequence's pitch, in place;
            # several: gathered (a few rows)
            cls = (lambda t: t[:, 0]) if n == 1 else (lambda t: t[:, :n].reshape(B * n, -1))
            gx_cls = g_x[:, 0] if n == 1 else torch.empty((B * n, Cin), dtype=x.dtype, device=x.device)
            kw = {"x_extra": cls(x), "gy_extra": cls(g_y), "gx_extra": gx_cls}
        _, g_W = _b.lbp_backward_ex(x[:, n:].unflatten(1, (H, W)), g_y[:, n:].unflatten(1, (H, W)),
                                    weight.contiguous(), ctx.k, ctx.bases, g_bias=g_b,
                                    gw_dtype=weight.dtype, g_x=g_x[:, n:].unflatten(1, (H, W)), **kw)
        if n > 1:
            g_x[:, :n] = gx_cls.view(B, n, Cin)
        return g_x, g_W, (None if g_b is None else g_b.to(weight.dtype)), None, None, None, None


class LbpLinear(torch.nn.Module):
    """Linear layer over a (B, H, W, C) token grid with LBP-WHT backward.

    `bases` is an ordered list of 0-based (i, j) sequency pairs, e.g. from
    `lbp_select_bases(k, SEL_L1, m)` (Eq. 8) or `lbp_select_lhe` (Sec. 3.2).
    """

    def __init__(self, in_features: int, out_features: int, k: int,
                 bases: Sequence[Tuple[int, int]], device=None, dtype=None, bias: bool = False,
                 save_projected: bool = False, grid=None):
        super().__init__()
        w = torch.empty((out_features, in_features), device=device, dtype=dtype)
        torch.nn.init.normal_(w, std=in_features ** -0.5)
        self.weight = torch.nn.Parameter(w)
        self.bias = (torch.nn.Parameter(torch.zeros(out_features, device=device, dtype=dtype))
                     if bias else None)
        self.k, self.bases = int(k), [tuple(p) for p in bases]
        self.save_projected = bool(save_projected)
        self.grid = None if grid is None else (int(grid[0]), int(grid[1]))

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return LbpLinearFunction.apply(x, self.weight, self.bias, self.k, self.bases,
                                       self.save_projected, self.grid)
