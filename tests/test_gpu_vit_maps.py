"""Parity of what a real ViT layer needs around Algorithm 1, against the oracle:
token grids whose sides are not multiples of the transform order (the paper's
own 7 x 7 maps of Sec. 3.3 and Table 5), tokens outside the grid (class token,
Eq. 2 exactly), the bias gradient, accumulation into g_W, and x_hat = p(x)
(Eq. 3) handed in instead of x.

Same bars as the other parity tests: relative Frobenius error 1e-5 (fp32) /
2e-2 (bf16) on whole outputs, 1e-5 / 1e-2 on the worst k x k block of g_x and the
worst 128 x 128 piece of g_W.
"""
import numpy as np
import pytest
import torch

import paper_2309_15275_b200 as lbp
import synth
from oracle import lbp_oracle as O

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-2}
LOCAL_TOL = {torch.float32: 1e-5, torch.bfloat16: 1e-2}


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


def rel(got, want):
    return O.rel_fro(f64(got), want)


def _layer(B, H, W, Cin, Cout, dtype, key):
    name = "f32" if dtype == torch.float32 else "bf16"
    x = synth.make_tensor((B, H, W, Cin), ("normal", 1.0), name, case_key=key, tensor_id=0)
    gy = synth.make_tensor((B, H, W, Cout), ("normal", 0.01), name, case_key=key, tensor_id=1)
    w = synth.make_tensor((Cout, Cin), ("normal", Cin ** -0.5), name, case_key=key, tensor_id=2)
    return x, gy, w


def _assert_grid_parity(gx, gw, ox, ow, k, dtype, what):
    assert rel(gx, ox) <= TOL[dtype], (what, "g_x")
    assert rel(gw, ow) <= TOL[dtype], (what, "g_W")
    # blocks of the zero-extended grid (the extension is zero on both sides)
    assert O.block_rel_fro(O.pad_grid(f64(gx), k), O.pad_grid(ox, k), k) <= LOCAL_TOL[dtype], what
    assert O.tile_rel_fro(f64(gw), ow, 128) <= LOCAL_TOL[dtype], what


# ------------------------------------------------ ragged grids: transforms ----
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k,H,W", [(8, 7, 7), (4, 7, 7), (8, 14, 14), (4, 14, 14), (16, 20, 33), (8, 9, 16)])
def test_project_expand_on_grids_that_are_no_multiple_of_k(dev, dtype, k, H, W):
    name = "f32" if dtype == torch.float32 else "bf16"
    t = synth.make_tensor((3, H, W, 200), ("normal", 1.0), name, case_key=1200 + k + H)
    for r in (1, 3, 10, min(21, k * k), k * k):
        bases = O.select_bases(k, O.RULE_PREFIX, r)
        got = lbp.lbp_project(t.to(dev), k, bases)
        want = O.project_padded(f64(t), k, bases)
        assert got.shape == want.shape
        assert rel(got, want) <= TOL[dtype], (k, r)
        th = torch.from_numpy(want).to(dtype)
        out = torch.full((3, H, W, 200), 7.0, dtype=dtype, device=dev)
        back = lbp.lbp_expand(th.to(dev), k, bases, out=out, grid=(H, W))
        want_back = O.expand(f64(th), k, bases)[:, :H, :W, :]
        assert rel(back, want_back) <= TOL[dtype], (k, r)
    # spectrum of the zero-extended grid: Parseval still holds on the real tokens
    e = lbp.lbp_spectrum(t.to(dev), k).cpu().numpy()
    want_e = O.spectrum(O.pad_grid(f64(t), k), k)
    assert np.max(np.abs(e - want_e) / want_e) <= (1e-5 if dtype == torch.float32 else 1e-4)


# -------------------------------- Table 5 workloads: (Cx, Cy, L = 49 tokens) ----
TABLE5 = [(448, 1792), (1792, 448), (768, 3072), (3072, 768)]


@pytest.mark.parametrize("Cin,Cout", TABLE5)
@pytest.mark.parametrize("k,H", [(8, 7), (4, 7), (8, 14), (4, 14)])
def test_table5_shapes_backward(dev, Cin, Cout, k, H):
    # LP_L1-2 / 4 / 6 (ranks 3, 10, 21) where the order has that many bases
    B = 32
    x, gy, w = _layer(B, H, H, Cin, Cout, torch.bfloat16, 1300 + H + k)
    xd, gd, wd = x.to(dev), gy.to(dev), w.to(dev)
    for m in (2, 4, 6):
        if m * (m + 1) // 2 > k * k:
            continue
        bases = O.select_bases(k, O.RULE_L1, m)
        gx, gw = lbp.lbp_backward(xd, gd, wd, k, bases)
        ox, ow = O.backward_lowrank_padded(f64(x), f64(gy), f64(w), k, bases)
        _assert_grid_parity(gx, gw, ox, ow, k, torch.bfloat16, (Cin, Cout, k, H, m))
    # all k*k bases: exact backpropagation on the real tokens
    gx, gw = lbp.lbp_backward(xd, gd, wd, k, O.select_bases(k, O.RULE_PREFIX, k * k))
    ex, ew = O.backward_exact(f64(x), f64(gy), f64(w))
    _assert_grid_parity(gx, gw, ex, ew, k, torch.bfloat16, (Cin, Cout, k, H, "full"))


def test_ragged_grid_fp32_and_rectangular(dev):
    x, gy, w = _layer(3, 10, 13, 40, 72, torch.float32, 1400)
    for k, r in ((4, 6), (8, 10), (8, 40), (16, 21)):
        bases = O.select_bases(k, O.RULE_PREFIX, r)
        gx, gw = lbp.lbp_backward(x.to(dev), gy.to(dev), w.to(dev), k, bases)
        ox, ow = O.backward_lowrank_padded(f64(x), f64(gy), f64(w), k, bases)
        _assert_grid_parity(gx, gw, ox, ow, k, torch.float32, (k, r))


@pytest.mark.parametrize("k,H,W,Cin,Cout,r", [(16, 20, 33, 256, 128, 6), (16, 17, 16, 64, 96, 16),
                                               (4, 9, 6, 192, 256, 7), (8, 15, 17, 128, 384, 36),
                                               (8, 7, 20, 64, 64, 21)])
def test_ragged_grid_bf16_on_the_products_kernels(dev, k, H, W, Cin, Cout, r):
    # edge blocks on both kernels of the persistent path (CTA pairs and one CTA),
    # every order, low and high rank
    x, gy, w = _layer(5, H, W, Cin, Cout, torch.bfloat16, 1450 + k + r)
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    gx, gw = lbp.lbp_backward(x.to(dev), gy.to(dev), w.to(dev), k, bases)
    ox, ow = O.backward_lowrank_padded(f64(x), f64(gy), f64(w), k, bases)
    _assert_grid_parity(gx, gw, ox, ow, k, torch.bfloat16, (k, H, W, r))


# ---------------- class token, bias gradient, accumulation (lbp_backward_ex) ----
@pytest.mark.parametrize("dtype,Cin,Cout,k,bases_kind", [
    (torch.bfloat16, 384, 768, 8, "l1_4"),        # products kernel on CTA pairs, DC selected
    (torch.bfloat16, 64, 192, 8, "l1_6"),         # separate kernels (r = 21)
    (torch.bfloat16, 256, 128, 4, "no_dc"),       # bias from g_y itself
    (torch.bfloat16, 256, 128, 8, "full"),        # full rank: Eq. 2, nothing materialised
    (torch.float32, 40, 72, 8, "l1_4"),
    (torch.float32, 40, 72, 4, "no_dc"),
])
def test_class_token_bias_and_accumulation(dev, dtype, Cin, Cout, k, bases_kind):
    B, H, W = 6, 14, 14
    x, gy, w = _layer(B, H, W, Cin, Cout, dtype, 1500 + Cin + k)
    name = "f32" if dtype == torch.float32 else "bf16"
    x_cls = synth.make_tensor((B, Cin), ("normal", 1.0), name, case_key=1501, tensor_id=3)
    gy_cls = synth.make_tensor((B, Cout), ("normal", 0.01), name, case_key=1501, tensor_id=4)
    gw_prev = synth.make_tensor((Cout, Cin), ("normal", 0.05), "f32", case_key=1501, tensor_id=5)
    gb_prev = synth.make_tensor((Cout,), ("normal", 0.5), "f32", case_key=1501, tensor_id=6)
    bases = {"l1_4": O.select_bases(k, O.RULE_L1, 4), "l1_6": O.select_bases(k, O.RULE_L1, 6),
             "no_dc": [(0, 1), (1, 0), (1, 1)],
             "full": O.select_bases(k, O.RULE_PREFIX, k * k)}[bases_kind]
    if bases_kind == "full":
        ox, ow = O.backward_exact(f64(x), f64(gy), f64(w))
    else:
        ox, ow = O.backward_lowrank_padded(f64(x), f64(gy), f64(w), k, bases)
    ox_cls, ow_cls = O.backward_extra_tokens(f64(x_cls), f64(gy_cls), f64(w))
    want_b = O.bias_grad(f64(gy), f64(gy_cls))

    for beta in (0.0, 1.0):
        g_W = gw_prev.clone().to(dev)
        g_b = gb_prev.clone().to(dev)
        gx_cls = torch.empty((B, Cin), dtype=dtype, device=dev)
        gx, _ = lbp.lbp_backward_ex(x.to(dev), gy.to(dev), w.to(dev), k, bases, beta=beta, g_bias=g_b,
                                    x_extra=x_cls.to(dev), gy_extra=gy_cls.to(dev), gx_extra=gx_cls,
                                    g_W=g_W)
        want_w = O.accumulate(ow + ow_cls, f64(gw_prev), beta)
        want_bias = O.accumulate(want_b, f64(gb_prev), beta)
        _assert_grid_parity(gx, g_W, ox, want_w, k, dtype, (bases_kind, beta))
        assert rel(gx_cls, ox_cls) <= TOL[dtype]
        assert rel(g_b, want_bias) <= TOL[dtype], (bases_kind, beta, "bias")
    # bias alone, no extra tokens, g_W overwritten
    g_b = torch.empty(Cout, dtype=torch.float32, device=dev)
    gx, gw = lbp.lbp_backward_ex(x.to(dev), gy.to(dev), w.to(dev), k, bases, g_bias=g_b)
    _assert_grid_parity(gx, gw, ox, ow, k, dtype, (bases_kind, "bias only"))
    assert rel(g_b, O.bias_grad(f64(gy))) <= TOL[dtype]


def test_extras_argument_errors(dev):
    x = torch.zeros((1, 8, 8, 64), dtype=torch.bfloat16, device=dev)
    gy = torch.zeros((1, 8, 8, 64), dtype=torch.bfloat16, device=dev)
    w = torch.zeros((64, 64), dtype=torch.bfloat16, device=dev)
    g_W = torch.full((64, 64), 3.0, device=dev)
    with pytest.raises(ValueError):      # both x and x_hat
        lbp.lbp_backward_ex(x, gy, w, 8, [(0, 0)], x_hat=torch.zeros((1, 1, 1, 1, 64), dtype=torch.bfloat16, device=dev))
    with pytest.raises(ValueError):      # a bias of the wrong type
        lbp.lbp_backward_ex(x, gy, w, 8, [(0, 0)], g_bias=torch.zeros(64, dtype=torch.bfloat16, device=dev))
    with pytest.raises(ValueError):      # W of another dtype would be read as bf16
        lbp.lbp_backward(x, gy, w.float(), 8, [(0, 0)])
    with pytest.raises(ValueError):      # W transposed / short
        lbp.lbp_backward(x, gy, torch.zeros((64, 32), dtype=torch.bfloat16, device=dev), 8, [(0, 0)])
    ws = torch.empty(lbp.lbp_workspace_bytes(1, 8, 8, 64, 64, 8, lbp.LBP_BF16, lbp.LBP_F32, 1),
                     dtype=torch.uint8, device=dev)
    assert lbp.lbp_workspace_bytes_ex(1, 8, 8, 64, 64, 8, lbp.LBP_BF16, lbp.LBP_F32, 1, beta=1.0) > ws.numel()
    with pytest.raises(lbp.LbpError) as e:   # the plain workspace is too small for accumulation
        lbp.lbp_backward_ex(x, gy, w, 8, [(0, 0)], beta=1.0, g_W=g_W, ws=ws)
    assert e.value.status == 7
    torch.cuda.synchronize()
    assert torch.all(g_W == 3.0)


# ------------------------------------- x_hat taken at forward time (Eq. 3) ----
@pytest.mark.parametrize("dtype,Cin,Cout,k,H,r", [
    (torch.bfloat16, 768, 768, 8, 16, 8),      # dense rows are the kernel's own layout
    (torch.bfloat16, 768, 384, 8, 16, 10),     # rows regrouped (128 is no multiple of 10)
    (torch.bfloat16, 256, 512, 8, 14, 3),      # ragged grid
    (torch.bfloat16, 64, 96, 4, 16, 5),        # one-CTA products kernel
    (torch.bfloat16, 128, 128, 8, 16, 21),     # separate kernels
    (torch.float32, 40, 72, 8, 16, 10),
    (torch.float32, 40, 72, 4, 8, 16),         # every basis, still through x_hat
])
def test_backward_from_projected_activation(dev, dtype, Cin, Cout, k, H, r):
    B = 8
    x, gy, w = _layer(B, H, H, Cin, Cout, dtype, 1600 + Cin + r)
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    # the coefficients come from the oracle, rounded once to the run dtype, and
    # both sides start from those bits
    x_hat = torch.from_numpy(O.project_padded(f64(x), k, bases)).to(dtype)
    gx, gw = lbp.lbp_backward_projected(x_hat.to(dev), gy.to(dev), w.to(dev), k, bases)
    ox, ow = O.backward_lowrank_projected(f64(x_hat), O.pad_grid(f64(gy), k), f64(w), k, bases)
    _assert_grid_parity(gx, gw, ox[:, :H, :H, :], ow, k, dtype, (Cin, Cout, k, r))
    # and it is Algorithm 1 on x, up to the rounding of x_hat
    fx, fw = O.backward_lowrank_padded(f64(x), f64(gy), f64(w), k, bases)
    assert rel(gx, fx) <= TOL[dtype] and rel(gw, fw) <= TOL[dtype]
    # the library's own projection feeds the same call
    th = lbp.lbp_project(x.to(dev), k, bases)
    gx2, gw2 = lbp.lbp_backward_projected(th, gy.to(dev), w.to(dev), k, bases)
    assert rel(gx2, fx) <= TOL[dtype] and rel(gw2, fw) <= TOL[dtype]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_autograd_layer_keeps_only_the_coefficients(dev, dtype):
    k, Cin, Cout = 8, 64, 96
    name = "f32" if dtype == torch.float32 else "bf16"
    x = synth.make_tensor((2, 14, 8, Cin), ("normal", 1.0), name, case_key=1700)
    gy = synth.make_tensor((2, 14, 8, Cout), ("normal", 1.0), name, case_key=1701)
    bases = O.select_bases(k, O.RULE_L1, 3)
    layer = lbp.LbpLinear(Cin, Cout, k, bases, device=dev, dtype=dtype, bias=True, save_projected=True)
    w = layer.weight.detach().clone()
    xd = x.to(dev).requires_grad_(True)
    y = layer(xd)
    saved = [t for t in y.grad_fn.saved_tensors] if hasattr(y.grad_fn, "saved_tensors") else []
    # what stays alive for the backward pass: r / k^2 of the activation (per padded block)
    assert any(t.shape == (2, 2, 1, len(bases), Cin) for t in saved)
    assert not any(t.shape == tuple(x.shape) for t in saved)
    y.backward(gy.to(dev))
    wx, ww = O.backward_lowrank_padded(f64(x), f64(gy), f64(w), k, bases)
    assert rel(xd.grad, wx) <= TOL[dtype]
    assert rel(layer.weight.grad, ww) <= TOL[dtype]
    assert rel(layer.bias.grad, O.bias_grad(f64(gy))) <= TOL[dtype]
