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


# ---------------------------------------------- views of larger tensors ----
@pytest.mark.parametrize("dtype,Cin,Cout,k,H,bases_kind", [
    (torch.bfloat16, 192, 256, 8, 14, "l1_4"),     # products kernel on CTA pairs, ragged grid
    (torch.bfloat16, 96, 64, 4, 7, "l1_2"),        # one-CTA products kernel
    (torch.bfloat16, 128, 128, 8, 14, "no_dc"),    # bias read from the strided g_y
    (torch.float32, 64, 96, 4, 7, "l1_2"),         # additions-only kernels, fp32
    (torch.bfloat16, 128, 192, 4, 8, "full"),      # Eq. 2 through dense copies
    (torch.float32, 64, 64, 4, 7, "full"),
])
def test_token_sequence_with_class_token_in_place(dev, dtype, Cin, Cout, k, H, bases_kind):
    # A ViT sequence (B, 1 + H*W, C): the grid tokens are a view behind the class
    # token (image stride (1 + H*W) * C), the class tokens rows with that pitch.
    # Nothing is copied by the caller; g_x lands in the sequence's own layout.
    B, W = 5, H
    name = "f32" if dtype == torch.float32 else "bf16"
    key = 2300 + Cin + k
    xs = synth.make_tensor((B, 1 + H * W, Cin), ("normal", 1.0), name, case_key=key, tensor_id=0)
    gys = synth.make_tensor((B, 1 + H * W, Cout), ("normal", 0.01), name, case_key=key, tensor_id=1)
    w = synth.make_tensor((Cout, Cin), ("normal", Cin ** -0.5), name, case_key=key, tensor_id=2)
    bases = {"l1_4": O.select_bases(k, O.RULE_L1, 4), "l1_2": O.select_bases(k, O.RULE_L1, 2),
             "no_dc": [(0, 1), (1, 0), (1, 1)],
             "full": O.select_bases(k, O.RULE_PREFIX, k * k)}[bases_kind]
    xg, gyg = xs[:, 1:].reshape(B, H, W, Cin), gys[:, 1:].reshape(B, H, W, Cout)   # dense copies for the oracle
    if bases_kind == "full":
        ox, ow = O.backward_exact(f64(xg), f64(gyg), f64(w))
    else:
        ox, ow = O.backward_lowrank_padded(f64(xg), f64(gyg), f64(w), k, bases)
    ox_cls, ow_cls = O.backward_extra_tokens(f64(xs[:, 0]), f64(gys[:, 0]), f64(w))
    want_b = O.bias_grad(f64(gyg), f64(gys[:, 0]))

    xd, gyd, wd = xs.to(dev), gys.to(dev), w.to(dev)
    gxs = torch.full((B, 1 + H * W, Cin), float("nan"), dtype=dtype, device=dev)
    g_b = torch.empty(Cout, dtype=torch.float32, device=dev)
    x_view = xd[:, 1:].unflatten(1, (H, W))
    gy_view = gyd[:, 1:].unflatten(1, (H, W))
    gx_view = gxs[:, 1:].unflatten(1, (H, W))
    assert not x_view.is_contiguous() and x_view.data_ptr() == xd.data_ptr() + Cin * xd.element_size()
    _, g_W = lbp.lbp_backward_ex(x_view, gy_view, wd, k, bases, g_bias=g_b, x_extra=xd[:, 0],
                                 gy_extra=gyd[:, 0], gx_extra=gxs[:, 0], g_x=gx_view)
    torch.cuda.synchronize()
    _assert_grid_parity(gxs[:, 1:].reshape(B, H, W, Cin), g_W, ox, ow + ow_cls, k, dtype, bases_kind)
    assert rel(gxs[:, 0], ox_cls) <= TOL[dtype]
    assert rel(g_b, want_b) <= TOL[dtype]
    # the same call on dense copies gives the same bits
    gx2 = torch.empty((B, H, W, Cin), dtype=dtype, device=dev)
    gxc2 = torch.empty((B, Cin), dtype=dtype, device=dev)
    g_b2 = torch.empty(Cout, dtype=torch.float32, device=dev)
    _, g_W2 = lbp.lbp_backward_ex(x_view.contiguous(), gy_view.contiguous(), wd, k, bases, g_bias=g_b2,
                                  x_extra=xd[:, 0].contiguous(), gy_extra=gyd[:, 0].contiguous(),
                                  gx_extra=gxc2, g_x=gx2)
    assert torch.equal(gxs[:, 1:].reshape(B, H, W, Cin), gx2) and torch.equal(gxs[:, 0], gxc2)
    assert torch.equal(g_W, g_W2) and torch.equal(g_b, g_b2)


@pytest.mark.parametrize("dtype,k,r", [(torch.bfloat16, 8, 8), (torch.float32, 4, 3), (torch.bfloat16, 8, 64)])
def test_channel_slices_of_wider_tensors(dev, dtype, k, r):
    # x, g_y and g_x are channel slices of wider tensors (token stride > C); what
    # lies beside the slice of g_x stays untouched.
    B, H, W, Cin, Cout = 3, 16, 24, 128, 192
    name = "f32" if dtype == torch.float32 else "bf16"
    x_big = synth.make_tensor((B, H, W, Cin + 64), ("normal", 1.0), name, case_key=2400 + k, tensor_id=0)
    gy_big = synth.make_tensor((B, H, W, 2 * Cout), ("normal", 0.01), name, case_key=2400 + k, tensor_id=1)
    w = synth.make_tensor((Cout, Cin), ("normal", Cin ** -0.5), name, case_key=2400 + k, tensor_id=2)
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    xs, gs = x_big[..., 32:32 + Cin], gy_big[..., Cout:]
    if r == k * k:
        ox, ow = O.backward_exact(f64(xs), f64(gs), f64(w))
    else:
        ox, ow = O.backward_lowrank(f64(xs), f64(gs), f64(w), k, bases)
    xd, gd = x_big.to(dev), gy_big.to(dev)
    gx_big = torch.full((B, H, W, Cin + 96), 7.0, dtype=dtype, device=dev)
    gx_view = gx_big[..., 64:64 + Cin]
    _, g_W = lbp.lbp_backward_ex(xd[..., 32:32 + Cin], gd[..., Cout:], w.to(dev), k, bases, g_x=gx_view)
    torch.cuda.synchronize()
    _assert_grid_parity(gx_view.contiguous(), g_W, ox, ow, k, dtype, ("slice", r))
    assert torch.all(gx_big[..., :64] == 7.0) and torch.all(gx_big[..., 64 + Cin:] == 7.0)


def test_view_argument_errors(dev):
    B, H, W, C = 2, 8, 8, 64
    x = torch.zeros((B, H, W, C + 4), dtype=torch.bfloat16, device=dev)
    gy = torch.zeros((B, H, W, C), dtype=torch.bfloat16, device=dev)
    w = torch.zeros((C, C), dtype=torch.bfloat16, device=dev)
    with pytest.raises((lbp.LbpError, ValueError)):     # token stride 68 elements: not 16-byte steps
        lbp.lbp_backward_ex(x[..., :C], gy, w, 8, [(0, 0)])
    with pytest.raises(ValueError):                     # channels not contiguous
        lbp.lbp_backward_ex(torch.zeros((B, H, C, W), dtype=torch.bfloat16, device=dev).transpose(2, 3),
                            gy, w, 8, [(0, 0)])
    # strides in the size query: a view adds the dense copies only in the full-rank mode
    base = lbp.lbp_workspace_bytes_ex(B, H, W, C, C, 8, lbp.LBP_BF16, lbp.LBP_F32, 8)
    v = (H * W * 2 * C, W * 2 * C, 2 * C)
    low = lbp.lbp_workspace_bytes_ex(B, H, W, C, C, 8, lbp.LBP_BF16, lbp.LBP_F32, 8, x_view=v)
    full0 = lbp.lbp_workspace_bytes_ex(B, H, W, C, C, 8, lbp.LBP_BF16, lbp.LBP_F32, 64)
    full = lbp.lbp_workspace_bytes_ex(B, H, W, C, C, 8, lbp.LBP_BF16, lbp.LBP_F32, 64, x_view=v)
    assert low >= base and full >= full0 + B * H * W * C * 2
    assert lbp.lbp_workspace_bytes_ex(B, H, W, C, C, 8, lbp.LBP_BF16, lbp.LBP_F32, 8,
                                      x_view=(H * W * C, W * C, C - 8)) == 0     # token stride < C


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


@pytest.mark.parametrize("n_cls", [1, 2])
def test_autograd_layer_on_a_token_sequence(dev, n_cls):
    # (B, n + H*W, C) as a ViT block hands it over: the class tokens take Eq. 2,
    # the grid tokens Algorithm 1, g_x comes back in the sequence's layout
    k, H, W, Cin, Cout, B = 8, 14, 14, 64, 128, 3
    dtype = torch.bfloat16
    x = synth.make_tensor((B, n_cls + H * W, Cin), ("normal", 1.0), "bf16", case_key=1710 + n_cls)
    gy = synth.make_tensor((B, n_cls + H * W, Cout), ("normal", 1.0), "bf16", case_key=1720 + n_cls)
    bases = O.select_bases(k, O.RULE_L1, 4)
    layer = lbp.LbpLinear(Cin, Cout, k, bases, device=dev, dtype=dtype, bias=True, grid=(H, W))
    w = layer.weight.detach().clone()
    xd = x.to(dev).requires_grad_(True)
    layer(xd).backward(gy.to(dev))
    xg, gyg = x[:, n_cls:].reshape(B, H, W, Cin), gy[:, n_cls:].reshape(B, H, W, Cout)
    xc, gyc = x[:, :n_cls].reshape(B * n_cls, Cin), gy[:, :n_cls].reshape(B * n_cls, Cout)
    wx, ww = O.backward_lowrank_padded(f64(xg), f64(gyg), f64(w), k, bases)
    wx_cls, ww_cls = O.backward_extra_tokens(f64(xc), f64(gyc), f64(w))
    assert rel(xd.grad[:, n_cls:].reshape(B, H, W, Cin), wx) <= TOL[dtype]
    assert rel(xd.grad[:, :n_cls].reshape(B * n_cls, Cin), wx_cls) <= TOL[dtype]
    assert rel(layer.weight.grad, ww + ww_cls) <= TOL[dtype]
    assert rel(layer.bias.grad, O.bias_grad(f64(gyg), f64(gyc))) <= TOL[dtype]
