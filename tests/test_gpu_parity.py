"""Parity of the CUDA path (through the C ABI) against the fp64 oracle.

Every comparison is on the same seeded inputs, already rounded to the run
dtype.  Bars: relative Frobenius error <= 1e-5 for fp32 data, <= 2e-2 for bf16
data with fp32 accumulation; basis lists bit-exact (checked on the CPU suite).

Beside the global bar every backward comparison has a local one, so that a
wrong patch cannot hide in the norm of a large tensor: the largest relative
Frobenius error over the k x k token blocks of g_x and over 128 x 128 pieces of
g_W.  For bf16 data the error is rounding noise of x_hat, g_y_hat and the
outputs to 8 mantissa bits (about 2^-9 per element, 2.4e-3 observed in the
norm of whole tensors); a block holds thousands of such elements, so its norm
ratio sits near the same figure, and the local bar is 1e-2, four times that.
A misplaced or dropped coefficient changes a block by the order of its norm.
"""
import functools
import os

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


def ok_status(ws):
    assert lbp.lbp_poll_status(ws) == 0


def coef_block_rel(got, want):
    """Largest relative error over the blocks of a coefficient tensor (B,Hb,Wb,r,C)."""
    d = f64(got) - want
    num = np.sqrt(np.sum(d * d, axis=(3, 4)))
    den = np.sqrt(np.sum(want * want, axis=(3, 4)))
    return float(np.max(np.where(den > 0, num / np.where(den > 0, den, 1.0), num)))


@functools.lru_cache(maxsize=2)
def _inputs(config, idx, batch):
    return synth.make_layer_inputs(synth.config_cases(config)[idx], batch=batch)


# ------------------------------------------------ projection / expansion ----
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k,ranks", [(4, (1, 2, 3, 5, 16)), (8, (1, 2, 4, 6, 8, 10, 16, 21, 36, 64)),
                                     (16, (1, 3, 8, 10, 36, 100, 256))])
def test_project_expand_prefix_sets(dev, dtype, k, ranks):
    # several blocks per image, ragged channel tail (C = 200 is not a multiple of a 128-byte chunk)
    B, Hb, Wb, C = 3, 2, 3, 200
    t = synth.make_tensor((B, Hb * k, Wb * k, C), ("normal", 1.0), "f32", case_key=700 + k).to(dtype)
    ws = torch.zeros(lbp.lbp_status_bytes(), dtype=torch.uint8, device=dev)
    for r in ranks:
        bases = O.select_bases(k, O.RULE_PREFIX, r)
        got = lbp.lbp_project(t.to(dev), k, bases, ws=ws)
        ok_status(ws)
        want = O.project(f64(t), k, bases)
        assert got.shape == want.shape
        assert rel(got, want) <= TOL[dtype], (k, r)
        assert coef_block_rel(got, want) <= LOCAL_TOL[dtype], (k, r)
        th = torch.from_numpy(want).to(dtype)
        back = lbp.lbp_expand(th.to(dev), k, bases, ws=ws)
        ok_status(ws)
        want_back = O.expand(f64(th), k, bases)
        assert rel(back, want_back) <= TOL[dtype], (k, r)
        assert O.block_rel_fro(f64(back), want_back, k) <= LOCAL_TOL[dtype], (k, r)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_project_arbitrary_sets_and_order(dev, dtype):
    k = 8
    t = synth.make_tensor((2, 16, 24, 72), ("normal", 1.0), "f32", case_key=710).to(dtype)
    for bases in ([(7, 0), (0, 7), (3, 3), (1, 6), (0, 0)], [(0, 1)], [(5, 5), (2, 0)],
                  list(reversed(O.select_bases(k, O.RULE_L1, 3))), O.select_bases(k, O.RULE_LINF, 3)):
        got = lbp.lbp_project(t.to(dev), k, bases)
        want = O.project(f64(t), k, bases)
        assert rel(got, want) <= TOL[dtype], bases
        th = torch.from_numpy(want).to(dtype)
        back = lbp.lbp_expand(th.to(dev), k, bases)
        assert rel(back, O.expand(f64(th), k, bases)) <= TOL[dtype], bases


def test_project_single_block_and_narrow_channels(dev):
    # H = W = k (one transform over the whole map), C narrower than one chunk
    for dtype, C in ((torch.bfloat16, 8), (torch.float32, 4), (torch.bfloat16, 48)):
        t = synth.make_tensor((1, 8, 8, C), ("normal", 1.0), "f32", case_key=720 + C).to(dtype)
        bases = O.select_bases(8, O.RULE_L1, 4)
        got = lbp.lbp_project(t.to(dev), 8, bases)
        assert rel(got, O.project(f64(t), 8, bases)) <= TOL[dtype]


def test_project_full_rank_is_lossless_fp32(dev):
    k = 8
    t = synth.make_tensor((2, 16, 16, 64), ("normal", 1.0), "f32", case_key=730)
    bases = O.select_bases(k, O.RULE_PREFIX, 64)
    th = lbp.lbp_project(t.to(dev), k, bases)
    back = lbp.lbp_expand(th, k, bases)
    assert rel(back, f64(t)) <= 1e-6


def test_argument_errors_leave_outputs_untouched(dev):
    t = torch.zeros((1, 8, 8, 8), dtype=torch.float32, device=dev)
    out = torch.full((1, 1, 1, 1, 8), 7.0, dtype=torch.float32, device=dev)
    ws = torch.zeros(256, dtype=torch.uint8, device=dev)
    for k, bases, status in ((8, [(0, 0), (0, 0)], 4), (8, [(8, 0)], 4), (5, [(0, 0)], 3)):
        with pytest.raises(lbp.LbpError) as e:
            lbp.lbp_project(t, k, bases, out=out, ws=ws)
        assert e.value.status == status
    with pytest.raises(lbp.LbpError) as e:      # an empty grid (no storage: a null pointer, too)
        lbp.lbp_project(torch.zeros((1, 0, 8, 8), device=dev), 8, [(0, 0)], out=out, ws=ws)
    assert e.value.status in (1, 2)
    with pytest.raises(lbp.LbpError) as e:      # C * 4 bytes not a multiple of 16
        lbp.lbp_project(torch.zeros((1, 8, 8, 6), device=dev), 8, [(0, 0)], out=out, ws=ws)
    assert e.value.status == 6
    with pytest.raises(lbp.LbpError) as e:      # workspace too small
        lbp.lbp_project(t, 8, [(0, 0)], out=out, ws=ws[:16])
    assert e.value.status == 7
    torch.cuda.synchronize()
    assert torch.all(out == 7.0)


# ------------------------------------------------------------ backward ----
def _run_backward(dev, case, r, batch=None, fullrank_entry=False, bases=None, idx=None):
    x, gy, w = _inputs(case.config, case.case_id if idx is None else idx, batch)
    k = case.k
    if bases is None:
        bases = O.select_bases(k, O.RULE_PREFIX, r)
    xd, gd, wd = x.to(dev), gy.to(dev), w.to(dev)
    ws = lbp.alloc_workspace(xd, gd, k, k * k if fullrank_entry else len(bases))
    if fullrank_entry:
        gx, gw = lbp.lbp_backward_fullrank(xd, gd, wd, k, ws=ws)
    else:
        gx, gw = lbp.lbp_backward(xd, gd, wd, k, bases, ws=ws)
    ok_status(ws)
    return (x, gy, w), bases, gx, gw


def _assert_parity(gx, gw, ox, ow, k, dtype, what):
    assert rel(gx, ox) <= TOL[dtype], (what, "g_x")
    assert rel(gw, ow) <= TOL[dtype], (what, "g_W")
    assert O.block_rel_fro(f64(gx), ox, k) <= LOCAL_TOL[dtype], (what, "g_x, worst block")
    assert O.tile_rel_fro(f64(gw), ow, 128) <= LOCAL_TOL[dtype], (what, "g_W, worst 128 x 128 piece")


def _check_lowrank(dev, case, r, batch=None, bases=None):
    (x, gy, w), bases, gx, gw = _run_backward(dev, case, r, batch, bases=bases)
    ox, ow = O.backward_lowrank(f64(x), f64(gy), f64(w), case.k, bases)
    _assert_parity(gx, gw, ox, ow, case.k, x.dtype, (case.name, r))


def test_config1_fp32(dev):
    case = synth.config_cases(1)[0]
    _check_lowrank(dev, case, 4)
    # full rank, through the generic entry and through the full-rank entry, equals exact BP
    x, gy, w = _inputs(1, 0, None)
    ex, ew = O.backward_exact(f64(x), f64(gy), f64(w))
    for entry in (False, True):
        _, _, gx, gw = _run_backward(dev, case, 64, fullrank_entry=entry)
        assert rel(gx, ex) <= 1e-5 and rel(gw, ew) <= 1e-5


@pytest.mark.parametrize("k,r", [(4, 3), (4, 9), (8, 10), (8, 40), (16, 6), (16, 130)])
def test_fp32_other_orders_and_ranks(dev, k, r):
    case = synth.LayerCase(1, f"fp32_k{k}", 2, 2 * k, 3 * k, 40, 72, k, (r,), "f32",
                           ("normal", 1.0), ("normal", 1.0), 3)
    x, gy, w = synth.make_layer_inputs(case)
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    gx, gw = lbp.lbp_backward(x.to(dev), gy.to(dev), w.to(dev), k, bases)
    ox, ow = O.backward_lowrank(f64(x), f64(gy), f64(w), k, bases)
    assert rel(gx, ox) <= 1e-5 and rel(gw, ow) <= 1e-5


@pytest.mark.parametrize("idx", [0, 1])
def test_config2_efficientformer_full_size(dev, idx):
    _check_lowrank(dev, synth.config_cases(2)[idx], 8)


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_config3_vitb_full_size(dev, idx):
    # every layer of the block at every rank of the configuration
    case = synth.config_cases(3)[idx]
    for r in (2, 4, 8, 16):
        _check_lowrank(dev, case, r)


@pytest.mark.parametrize("switch", ["LBP_PAIR", "LBP_FUSED", "LBP_PROJECT_UMMA"])
def test_config3_through_the_switched_paths(dev, switch):
    # LBP_PAIR=0: the one-CTA products kernel on wide layers; LBP_FUSED=0: separate
    # product and expansion kernels; LBP_PROJECT_UMMA=0: order-8 projection on warp
    # mma.sync instead of tcgen05.  Same bars as the default path.
    os.environ[switch] = "0"
    lbp.lbp_test_reload_env()
    try:
        for idx in (1, 2):
            _check_lowrank(dev, synth.config_cases(3)[idx], 8)
        if switch == "LBP_PROJECT_UMMA":
            # the warp-level kernels at the ranks and orders the tcgen05 kernel takes by default
            _check_lowrank(dev, synth.config_cases(5)[1], 36, batch=2)
            _check_lowrank(dev, synth.config_cases(5)[2], 36, batch=2)
            _check_lowrank(dev, synth.config_cases(5)[2], 21, batch=2)
    finally:
        del os.environ[switch]
        lbp.lbp_test_reload_env()


@pytest.mark.parametrize("idx", [0, 1])
def test_config4_vitl_full_size(dev, idx):
    _check_lowrank(dev, synth.config_cases(4)[idx], 6)


def test_bf16_ragged_rows_and_small_batches(dev):
    # M_hat not a multiple of the 128-row MMA tile, K not a multiple of 64
    case = synth.config_cases(3)[1]
    for batch, r in ((1, 3), (3, 10), (5, 21)):
        _check_lowrank(dev, case, r, batch=batch)
    odd = synth.LayerCase(3, "odd", 3, 16, 24, 200, 328, 8, (5,), "bf16",
                          ("normal", 1.0), ("normal", 0.01), 9)
    x, gy, w = synth.make_layer_inputs(odd)
    bases = O.select_bases(8, O.RULE_L1, 3)
    gx, gw = lbp.lbp_backward(x.to(dev), gy.to(dev), w.to(dev), 8, bases)
    ox, ow = O.backward_lowrank(f64(x), f64(gy), f64(w), 8, bases)
    assert rel(gx, ox) <= 2e-2 and rel(gw, ow) <= 2e-2


def test_bf16_gw_in_bf16(dev):
    case = synth.config_cases(3)[1]
    x, gy, w = _inputs(3, 1, 8)
    bases = O.select_bases(8, O.RULE_PREFIX, 8)
    gx, gw = lbp.lbp_backward(x.to(dev), gy.to(dev), w.to(dev), 8, bases, gw_dtype=torch.bfloat16)
    assert gw.dtype == torch.bfloat16
    ox, ow = O.backward_lowrank(f64(x), f64(gy), f64(w), 8, bases)
    assert rel(gx, ox) <= 2e-2 and rel(gw, ow) <= 2e-2


def test_bf16_full_rank_is_exact_bp(dev):
    case = synth.config_cases(3)[1]
    x, gy, w = _inputs(3, 1, 16)
    ex, ew = O.backward_exact(f64(x), f64(gy), f64(w))
    for entry in (False, True):
        _, _, gx, gw = _run_backward(dev, case, 64, batch=16, fullrank_entry=entry)
        assert rel(gx, ex) <= 2e-2 and rel(gw, ew) <= 2e-2


# ranks chosen so that every expansion variant of the products kernel (cores of
# 1, 2, 4 and 8 coefficients per side, the 4 x 4 core plus one or two extra
# bases at r = 14..16, ranks up to 48 at orders 8 and 16), the generic path and the full-rank mode run at
# full size
@pytest.mark.parametrize("idx,ranks", [(0, (1, 2, 4, 7, 12, 16)),
                                       (1, (1, 2, 3, 5, 8, 11, 12, 13, 14, 15, 21, 28, 32, 36, 48, 50, 64)),
                                       (2, (1, 3, 5, 10, 14, 16, 17, 21, 32, 36, 48, 49, 100, 256))])
def test_config5_sweep_full_size(dev, idx, ranks):
    case = synth.config_cases(5)[idx]
    for r in ranks:
        if r == case.k * case.k:
            (x, gy, w), _, gx, gw = _run_backward(dev, case, r)
            ex, ew = O.backward_exact(f64(x), f64(gy), f64(w))
            _assert_parity(gx, gw, ex, ew, case.k, x.dtype, (case.name, "full rank"))
        else:
            _check_lowrank(dev, case, r)


def test_outputs_do_not_depend_on_basis_order(dev):
    case = synth.config_cases(3)[1]
    x, gy, w = _inputs(3, 1, 4)
    bases = O.select_bases(8, O.RULE_L1, 3)
    perm = [bases[i] for i in (3, 0, 5, 1, 4, 2)]
    a = lbp.lbp_backward(x.to(dev), gy.to(dev), w.to(dev), 8, bases)
    b = lbp.lbp_backward(x.to(dev), gy.to(dev), w.to(dev), 8, perm)
    ox, ow = O.backward_lowrank(f64(x), f64(gy), f64(w), 8, bases)
    for got in (a, b):
        _assert_parity(got[0], got[1], ox, ow, 8, x.dtype, "order")
    # the order only permutes the rows of x_hat / g_y_hat: the sums of g_W are taken
    # in another order (fp32), g_x sees the same arithmetic
    assert rel(b[1], f64(a[1])) <= 1e-5 and rel(b[0], f64(a[0])) <= 1e-3


def test_repeated_calls_are_deterministic(dev):
    case = synth.config_cases(3)[1]
    x, gy, w = _inputs(3, 1, 8)
    bases = O.select_bases(8, O.RULE_PREFIX, 8)
    xd, gd, wd = x.to(dev), gy.to(dev), w.to(dev)
    a = lbp.lbp_backward(xd, gd, wd, 8, bases)
    b = lbp.lbp_backward(xd, gd, wd, 8, bases)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


# ------------------------------------------ LHE profiling (Sec. 3.2) ----
def _low_frequency_tensor(shape, k, dtype, key):
    """Noise plus a strong block-smooth part: most energy in the low responses,
    as the paper reports for real gradients (Sec. 4, spectrum figure)."""
    B, H, W, C = shape
    fine = synth.make_tensor(shape, ("normal", 0.25), "f32", case_key=key)
    coarse = synth.make_tensor((B, H // 2, W // 2, C), ("normal", 1.0), "f32", case_key=key + 1)
    smooth = coarse.repeat_interleave(2, dim=1).repeat_interleave(2, dim=2)
    return (fine + smooth).to(dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k", [4, 8, 16])
def test_spectrum_matches_oracle(dev, dtype, k):
    shape = (3, 2 * k, 3 * k, 200)   # several blocks, ragged channel tail
    t = _low_frequency_tensor(shape, k, dtype, 900 + k)
    e = lbp.lbp_spectrum(t.to(dev), k)
    want = O.spectrum(f64(t), k)
    got = e.cpu().numpy()
    assert got.shape == (k, k)
    # Every energy on its own, so that the weak responses (the ones a selection
    # ranks) are held to the same bar as the DC term.  fp32 data: coefficients and
    # sums in fp32.  bf16 data: the +-1 products of bf16 values are exact, sums in
    # fp32 / fp64, nothing is rounded to bf16 on the way.
    tol = 1e-5 if dtype == torch.float32 else 1e-4
    assert np.max(np.abs(got - want) / want) <= tol
    assert abs(got.sum() - np.sum(f64(t) ** 2)) <= tol * np.sum(f64(t) ** 2)   # Parseval
    # the selection is taken on the host from the energies: same list wherever
    # the oracle's energies are separated by more than the tolerance
    for r in (1, 4, k):
        sel = lbp.lbp_select_lhe(got, k, r)
        ref = O.select_lhe(want, k, r)
        srt = np.sort(want.ravel())[::-1]
        if r < k * k and (srt[r - 1] - srt[r]) > 4 * tol * srt[r - 1]:
            assert set(sel) == set(ref)
        assert sel == O.select_lhe(got, k, r)
    # second call into the same output: overwritten, not accumulated
    e2 = lbp.lbp_spectrum(t.to(dev), k, out=e)
    assert np.allclose(e2.cpu().numpy(), got, rtol=1e-12)


def test_spectrum_full_size_layer_and_lhe_backward(dev):
    # g_y of the ViT-B qkv layer at full size; then Algorithm 1 on the selected bases
    case = synth.config_cases(3)[0]
    x, gy, w = _inputs(3, 0, None)
    k = case.k
    e = lbp.lbp_spectrum(gy.to(dev), k).cpu().numpy()
    total = float(torch.sum(gy.to(dev).double() ** 2))
    assert abs(e.sum() - total) <= 2e-2 * total
    # sampled check against the oracle: 8 images
    want = O.spectrum(f64(gy[:8]), k)
    got8 = lbp.lbp_spectrum(gy[:8].contiguous().to(dev), k).cpu().numpy()
    assert np.max(np.abs(got8 - want) / want) <= 1e-4
    bases = lbp.lbp_select_lhe(e, k, 8)
    assert len(set(bases)) == 8
    xs, gs = x[:4].contiguous(), gy[:4].contiguous()
    g_x, g_W = lbp.lbp_backward(xs.to(dev), gs.to(dev), w.to(dev), k, bases)
    wx, ww = O.backward_lowrank(f64(xs), f64(gs), f64(w), k, bases)
    assert rel(g_x, wx) <= 2e-2 and rel(g_W, ww) <= 2e-2


def test_spectrum_argument_errors(dev):
    t = torch.zeros((1, 8, 8, 64), dtype=torch.bfloat16, device=dev)
    e = torch.full((8, 8), -1.0, dtype=torch.float64, device=dev)
    with pytest.raises(lbp.LbpError) as err:
        lbp.lbp_spectrum(t, 8, out=e, ws=torch.zeros(256, dtype=torch.uint8, device=dev))
    assert err.value.status == 7 and float(e.min()) == -1.0
    with pytest.raises(ValueError):
        lbp.lbp_spectrum(torch.zeros((1, 8, 12, 60), dtype=torch.bfloat16, device=dev), 8)


# ------------------------------------------------ autograd front end ----
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_autograd_linear_backward_is_algorithm_1(dev, dtype):
    k, Cin, Cout = 8, 64, 96
    name = "f32" if dtype == torch.float32 else "bf16"
    x = synth.make_tensor((2, 16, 8, Cin), ("normal", 1.0), name, case_key=950)
    gy = synth.make_tensor((2, 16, 8, Cout), ("normal", 1.0), name, case_key=951)
    bases = O.select_bases(k, O.RULE_L1, 3)
    layer = lbp.LbpLinear(Cin, Cout, k, bases, device=dev, dtype=dtype)
    w = layer.weight.detach().clone()
    xd = x.to(dev).requires_grad_(True)
    y = layer(xd)
    want_y = f64(x) @ f64(w).T
    assert rel(y.detach(), want_y) <= TOL[dtype]
    y.backward(gy.to(dev))
    wx, ww = O.backward_lowrank(f64(x), f64(gy), f64(w), k, bases)
    assert rel(xd.grad, wx) <= TOL[dtype]
    assert rel(layer.weight.grad, ww) <= TOL[dtype]
    assert layer.weight.grad.dtype == dtype


# ------------------------------------------------------ batch of layers ----
def test_batch_equals_single_calls_and_rejects_overlap(dev):
    k, r = 8, 8
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    shapes = [(768, 2304), (768, 768), (256, 1024), (64, 64)]   # the last one takes the narrow-layer kernel
    xs, gys, ws_, singles = [], [], [], []
    for n, (ci, co) in enumerate(shapes):
        x = synth.make_tensor((4, 16, 16, ci), ("normal", 1.0), "bf16", case_key=960 + n).to(dev)
        gy = synth.make_tensor((4, 16, 16, co), ("normal", 0.01), "bf16", case_key=970 + n).to(dev)
        w = synth.make_tensor((co, ci), ("normal", ci ** -0.5), "bf16", case_key=980 + n).to(dev)
        xs.append(x), gys.append(gy), ws_.append(w)
        singles.append(lbp.lbp_backward(x, gy, w, k, bases))
    g_xs = [torch.empty_like(x) for x in xs]
    g_Ws = [torch.empty((w.shape[0], w.shape[1]), dtype=torch.float32, device=dev) for w in ws_]
    wss = [lbp.alloc_workspace(x, gy, k, r) for x, gy in zip(xs, gys)]
    for _ in range(2):
        lbp.lbp_backward_batch(xs, gys, ws_, k, bases, g_xs=g_xs, g_Ws=g_Ws, wss=wss)
    for i in range(len(shapes)):
        ok_status(wss[i])
        assert torch.equal(g_xs[i], singles[i][0]) and torch.equal(g_Ws[i], singles[i][1])
    # against the oracle too (the narrow layer)
    wx, ww = O.backward_lowrank(f64(xs[3]), f64(gys[3]), f64(ws_[3]), k, bases)
    assert rel(g_xs[3], wx) <= 2e-2 and rel(g_Ws[3], ww) <= 2e-2
    # an output of one problem that is an input of another is refused before any launch
    before = g_xs[1].clone()
    with pytest.raises(lbp.LbpError) as err:
        lbp.lbp_backward_batch([xs[0], g_xs[0]], [gys[0], gys[1]], [ws_[0], ws_[1]], k, bases,
                               g_xs=[g_xs[0], g_xs[1]], g_Ws=[g_Ws[0], g_Ws[1]], wss=[wss[0], wss[1]])
    assert err.value.status == 12
    with pytest.raises(lbp.LbpError) as err:   # shared workspace
        lbp.lbp_backward_batch(xs[:2], gys[:2], ws_[:2], k, bases, g_xs=g_xs[:2], g_Ws=g_Ws[:2],
                               wss=[wss[0], wss[0]])
    assert err.value.status in (7, 12)
    torch.cuda.synchronize()
    assert torch.equal(g_xs[1], before)


def test_batch_of_wide_layers_runs_beside_each_other(dev):
    # every layer takes the products kernel on CTA pairs: the batch call runs the
    # projection of one beside the products kernel of another (its own stream,
    # its own order) and records an event per layer.  g_x has one summation order
    # whatever the tile plan; g_W may be summed in other K slices than in a
    # single call, so it is compared within fp32 rounding, and with the oracle.
    k, r = 8, 8
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    shapes = [(768, 768), (256, 1024), (1024, 256), (384, 384)]
    xs, gys, ws_, singles = [], [], [], []
    for n, (ci, co) in enumerate(shapes):
        x = synth.make_tensor((8, 16, 16, ci), ("normal", 1.0), "bf16", case_key=1960 + n).to(dev)
        gy = synth.make_tensor((8, 16, 16, co), ("normal", 0.01), "bf16", case_key=1970 + n).to(dev)
        w = synth.make_tensor((co, ci), ("normal", ci ** -0.5), "bf16", case_key=1980 + n).to(dev)
        xs.append(x), gys.append(gy), ws_.append(w)
        singles.append(lbp.lbp_backward(x, gy, w, k, bases))
    g_xs = [torch.empty_like(x) for x in xs]
    g_Ws = [torch.empty((w.shape[0], w.shape[1]), dtype=torch.float32, device=dev) for w in ws_]
    wss = [lbp.alloc_workspace(x, gy, k, r) for x, gy in zip(xs, gys)]
    events = [torch.cuda.Event() for _ in shapes]
    side = torch.cuda.Stream(device=dev)
    sums = []
    for _ in range(3):
        for g in g_xs + g_Ws:
            g.fill_(float("nan"))
        lbp.lbp_backward_batch(xs, gys, ws_, k, bases, g_xs=g_xs, g_Ws=g_Ws, wss=wss, done_events=events)
        # a consumer on another stream, behind each layer's event
        with torch.cuda.stream(side):
            cur = []
            for e, g in zip(events, g_Ws):
                side.wait_event(e)
                cur.append(g.double().sum())
        torch.cuda.current_stream().wait_stream(side)
        sums.append([float(v) for v in cur])
    for i in range(len(shapes)):
        ok_status(wss[i])
        assert torch.equal(g_xs[i], singles[i][0])
        assert rel(g_Ws[i], f64(singles[i][1])) <= 1e-6
        assert sums[0][i] == sums[1][i] == sums[2][i] == float(g_Ws[i].double().sum())   # complete at the event, and deterministic
    wx, ww = O.backward_lowrank(f64(xs[1]), f64(gys[1]), f64(ws_[1]), k, bases)
    _assert_parity(g_xs[1], g_Ws[1], wx, ww, k, torch.bfloat16, "batch, side stream")


def test_batch_call_replays_from_a_cuda_graph(dev):
    # The whole block (four layers, projections on the library's stream beside the
    # products kernels) captured once and replayed: the replay must give what the
    # direct call gives, also after the inputs changed in place.
    k, r = 8, 8
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    shapes = [(768, 768), (256, 1024), (1024, 256), (384, 384)]
    xs, gys, ws_ = [], [], []
    for n, (ci, co) in enumerate(shapes):
        xs.append(synth.make_tensor((8, 16, 16, ci), ("normal", 1.0), "bf16", case_key=2060 + n).to(dev))
        gys.append(synth.make_tensor((8, 16, 16, co), ("normal", 0.01), "bf16", case_key=2070 + n).to(dev))
        ws_.append(synth.make_tensor((co, ci), ("normal", ci ** -0.5), "bf16", case_key=2080 + n).to(dev))
    wss = [lbp.alloc_workspace(x, gy, k, r) for x, gy in zip(xs, gys)]

    def outputs():
        return ([torch.full_like(x, float("nan")) for x in xs],
                [torch.full((w.shape[0], w.shape[1]), float("nan"), dtype=torch.float32, device=dev)
                 for w in ws_])

    def direct():
        g_xs, g_Ws = outputs()
        lbp.lbp_backward_batch(xs, gys, ws_, k, bases, g_xs=g_xs, g_Ws=g_Ws, wss=wss)
        torch.cuda.synchronize()
        return g_xs, g_Ws

    want = direct()     # also the first call: the library makes its stream and events here
    g_xs, g_Ws = outputs()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        lbp.lbp_backward_batch(xs, gys, ws_, k, bases, g_xs=g_xs, g_Ws=g_Ws, wss=wss)
    for rep in range(2):
        for g in g_xs + g_Ws:
            g.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        for i in range(len(shapes)):
            ok_status(wss[i])
            assert torch.equal(g_xs[i], want[0][i]) and torch.equal(g_Ws[i], want[1][i]), (rep, i)
    # new values in the same buffers
    for n, x in enumerate(xs):
        x.copy_(synth.make_tensor(tuple(x.shape), ("normal", 1.0), "bf16", case_key=2090 + n).to(dev))
    graph.replay()
    torch.cuda.synchronize()
    want = direct()
    for i in range(len(shapes)):
        assert torch.equal(g_xs[i], want[0][i]) and torch.equal(g_Ws[i], want[1][i]), i
    ex, ew = O.backward_lowrank(f64(xs[0]), f64(gys[0]), f64(ws_[0]), k, bases)
    _assert_parity(g_xs[0], g_Ws[0], ex, ew, k, torch.bfloat16, "graph replay")
