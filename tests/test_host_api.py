"""CPU-side checks of the C ABI: the library loads, exports every declared
symbol, and its host-only functions agree with the oracle bit for bit."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2309_15275_b200 as lbp
from oracle import lbp_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2309_15275_b200.build import build_library
    build_library()


def test_library_exports_every_declared_symbol():
    inc = os.path.join(ROOT, "include")
    header = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    declared = set(re.findall(r"^(?:int|size_t|double|long long|const char\*)\s+(lbp_[a-z_]+)\s*\(", header, re.M))
    assert declared == set(lbp.EXPORTED)
    lib = ctypes.CDLL(lbp.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("k", (4, 8, 16))
def test_select_bases_bit_exact_vs_oracle(k):
    for m in range(1, 2 * k):
        assert lbp.lbp_select_bases(k, lbp.SEL_L1, m) == O.select_bases(k, O.RULE_L1, m)
    for m in range(1, k + 1):
        assert lbp.lbp_select_bases(k, lbp.SEL_LINF, m) == O.select_bases(k, O.RULE_LINF, m)
    for r in range(1, k * k + 1):
        assert lbp.lbp_select_bases(k, lbp.SEL_PREFIX, r) == O.select_bases(k, O.RULE_PREFIX, r)


@pytest.mark.parametrize("k", (4, 8, 16))
def test_basis_matrix_bit_exact_vs_oracle(k):
    rng = np.random.default_rng(k)
    for r in (1, 3, k, k * k):
        pairs = [(int(p) // k, int(p) % k) for p in rng.permutation(k * k)[:r]]
        assert np.array_equal(lbp.lbp_basis_matrix(k, pairs), O.basis_matrix(k, pairs))


def test_flops_match_table1():
    f = O.flops(3072, 768, 49, 8)
    assert lbp.lbp_flops(3072, 768, 49, 8, 0) == f["vanilla"]
    assert lbp.lbp_flops(3072, 768, 49, 8, 1) == f["projection"]
    assert lbp.lbp_flops(3072, 768, 49, 8, 2) == f["lowrank_mm"]
    assert lbp.lbp_flops(3072, 768, 49, 8, 3) == f["reverse_projection"]
    assert lbp.lbp_flops(3072, 768, 49, 8, 4) == f["projection"] + f["lowrank_mm"] + f["reverse_projection"]
    assert lbp.lbp_flops(1, 1, 1, 1, 9) < 0


def test_argument_errors():
    with pytest.raises(lbp.LbpError) as e:
        lbp.lbp_select_bases(5, lbp.SEL_L1, 2)
    assert e.value.status == 3
    with pytest.raises(lbp.LbpError) as e:
        lbp.lbp_select_bases(8, lbp.SEL_PREFIX, 65)
    assert e.value.status == 4
    with pytest.raises(lbp.LbpError) as e:
        lbp.lbp_basis_matrix(8, [(0, 0), (0, 0)])
    assert e.value.status == 4
    with pytest.raises(lbp.LbpError) as e:
        lbp.lbp_basis_matrix(8, [(0, 8)])
    assert e.value.status == 4
    assert "basis" in lbp.lbp_status_string(4)


def test_workspace_bytes():
    n8 = lbp.lbp_workspace_bytes(128, 16, 16, 768, 3072, 8, lbp.LBP_BF16, lbp.LBP_F32, 8)
    n16 = lbp.lbp_workspace_bytes(128, 16, 16, 768, 3072, 8, lbp.LBP_BF16, lbp.LBP_F32, 16)
    rows = 512 * 8
    assert n8 >= rows * (768 + 3072) * 2 + rows * 768 * 4
    assert n16 > n8
    # a grid side that is no multiple of k is extended with zero tokens: as many blocks as 16 x 16
    assert (lbp.lbp_workspace_bytes(128, 16, 12, 768, 3072, 8, lbp.LBP_BF16, lbp.LBP_F32, 8)
            == lbp.lbp_workspace_bytes(128, 16, 16, 768, 3072, 8, lbp.LBP_BF16, lbp.LBP_F32, 8))
    assert lbp.lbp_workspace_bytes(128, 16, 0, 768, 3072, 8, lbp.LBP_BF16, lbp.LBP_F32, 8) == 0
    assert lbp.lbp_workspace_bytes(128, 16, 16, 768, 3072, 8, lbp.LBP_F32, lbp.LBP_BF16, 8) == 0   # dtype combo
    assert lbp.lbp_workspace_bytes(128, 16, 16, 768, 3072, 8, lbp.LBP_BF16, lbp.LBP_F32, 65) == 0


def test_device_calls_fail_loudly_without_cuda_tensors():
    import torch
    t = torch.zeros((1, 8, 8, 8), dtype=torch.float32)
    with pytest.raises(ValueError):
        lbp.lbp_project(t, 8, [(0, 0)], out=torch.zeros((1, 1, 1, 1, 8)), ws=torch.zeros(256, dtype=torch.uint8))


@pytest.mark.parametrize("k", (4, 8, 16))
def test_select_lhe_bit_exact_vs_oracle(k):
    rng = np.random.default_rng(40 + k)
    # distinct energies, then a quantised array with many ties
    for energy in (rng.random((k, k)), np.round(rng.random((k, k)) * 4) / 4):
        for r in (1, 2, k, k * k // 2, k * k):
            assert lbp.lbp_select_lhe(energy, k, r) == O.select_lhe(energy, k, r)


def test_select_lhe_argument_errors():
    e = np.ones((8, 8))
    for bad_r in (0, 65):
        with pytest.raises(lbp.LbpError) as err:
            lbp.lbp_select_lhe(e, 8, bad_r)
        assert err.value.status == 4
    bad = e.copy()
    bad[1, 1] = -1.0
    with pytest.raises(lbp.LbpError) as err:
        lbp.lbp_select_lhe(bad, 8, 3)
    assert err.value.status == 4
    bad[1, 1] = float("nan")
    with pytest.raises(lbp.LbpError) as err:
        lbp.lbp_select_lhe(bad, 8, 3)
    assert err.value.status == 4
    with pytest.raises(lbp.LbpError) as err:
        lbp.lbp_select_lhe(np.ones((5, 5)), 5, 3)
    assert err.value.status == 3
    assert lbp.lbp_spectrum_workspace_bytes(2, 16, 16, 64, 8, lbp.LBP_BF16) >= 2 * 16 * 16 * 64 * 2
    assert (lbp.lbp_spectrum_workspace_bytes(2, 15, 16, 64, 8, lbp.LBP_BF16)
            == lbp.lbp_spectrum_workspace_bytes(2, 16, 16, 64, 8, lbp.LBP_BF16))
    assert lbp.lbp_spectrum_workspace_bytes(2, 15, 16, 60, 8, lbp.LBP_BF16) == 0


def test_batch_arguments_are_checked_on_the_host_before_any_device_call():
    # fake (never dereferenced) device addresses: every check below happens on the
    # host, before the library touches the CUDA runtime
    from paper_2309_15275_b200 import binding as b
    lib = b._lib()
    n, k, r = 2, 8, 8
    bases = lbp.lbp_select_bases(k, lbp.SEL_PREFIX, r)
    lays = (b.Layer * n)(b._layer(2, 16, 16, 64, 128, k, lbp.LBP_BF16, lbp.LBP_F32),
                         b._layer(2, 16, 16, 128, 64, k, lbp.LBP_BF16, lbp.LBP_F32))
    need = [lbp.lbp_workspace_bytes(2, 16, 16, 64, 128, k, lbp.LBP_BF16, lbp.LBP_F32, r),
            lbp.lbp_workspace_bytes(2, 16, 16, 128, 64, k, lbp.LBP_BF16, lbp.LBP_F32, r)]
    MB = 1 << 20
    base = 1 << 32

    def arr(vals):
        return (ctypes.c_void_p * n)(*vals)

    def call(x, gy, w, gx, gw, ws, sizes=None):
        sz = (ctypes.c_size_t * n)(*(sizes or need))
        return lib.lbp_backward_batch(n, arr(x), arr(gy), arr(w), arr(gx), arr(gw), lays,
                                      b._bases(bases), r, arr(ws), sz, None, None)

    x = [base, base + 64 * MB]
    gy = [base + 8 * MB, base + 72 * MB]
    w = [base + 16 * MB, base + 80 * MB]
    gx = [base + 24 * MB, base + 88 * MB]
    gw = [base + 32 * MB, base + 96 * MB]
    ws = [base + 40 * MB, base + 104 * MB]
    # g_x of problem 0 is x of problem 1
    assert call([x[0], gx[0]], gy, w, gx, gw, ws) == 12
    # the two problems share an output
    assert call(x, gy, w, gx, [gw[0], gw[0]], ws) == 12
    # workspace of problem 1 overlaps g_y of problem 0
    assert call(x, gy, w, gx, gw, [ws[0], gy[0]]) == 12
    # shared inputs are allowed: the next check that fails is the workspace size
    assert call([x[0], x[0] + 0], gy, [w[0], w[0]], gx, gw, ws, sizes=[need[0], 16]) in (2, 7)
    assert call(x, gy, w, gx, gw, ws, sizes=[need[0], need[1] - 1]) == 7
    assert call(x, gy, w, [gx[0], gx[1] + 2], gw, ws) == 6          # misaligned pointer
    assert call(x, gy, w, [gx[0], None], gw, ws) == 1               # null pointer
    assert lib.lbp_backward_batch(0, arr(x), arr(gy), arr(w), arr(gx), arr(gw), lays,
                                  b._bases(bases), r, arr(ws), (ctypes.c_size_t * n)(*need), None, None) == 2
    assert "overlap" in lbp.lbp_status_string(12)


@pytest.mark.parametrize("Cin,Cout,G,bpt,units,pair", [
    (768, 2304, 32, 16, 74, 1), (768, 768, 32, 16, 74, 1), (768, 3072, 32, 16, 74, 1),
    (3072, 768, 32, 16, 74, 1), (1024, 4096, 25, 21, 74, 1), (48, 192, 196, 16, 148, 0),
    (192, 48, 196, 16, 148, 0), (64, 64, 1, 4, 148, 0), (768, 3072, 5, 2, 66, 1)])
def test_tile_plan_covers_every_tile_once(Cin, Cout, G, bpt, units, pair):
    # what the products kernel is told to do: every tile of both products exactly
    # once, GX tiles (long epilogue) ahead of GW tiles on every unit
    max_splits = 8
    info, lists = lbp.lbp_test_tile_plan(Cin, Cout, G, bpt, 8, units, pair, max_splits)
    row_tile = 256 if pair else 128
    step = 128 if pair else 64
    assert info["BNw"] % step == 0 and info["BNx"] % step == 0 and info["BNw"] <= 256 and info["BNx"] <= 256
    assert 1 <= info["splits"] <= max_splits
    assert info["kbps"] * info["splits"] >= 2 * G > info["kbps"] * (info["splits"] - 1)
    n_gw = -(-Cout // row_tile) * -(-Cin // info["BNw"]) * info["splits"]
    n_gx = (-(-G // 2) if pair else G) * -(-Cin // info["BNx"])
    assert info["listed"] and lists is not None
    flat = [t for unit in lists for t in unit]
    assert sorted(flat) == list(range(n_gw + n_gx))
    for unit in lists:
        kinds = [t < n_gw for t in unit]            # True = GW
        assert kinds == sorted(kinds)               # all GX tiles first
    # no unit is left without work while another holds three tiles more
    sizes = [len(u) for u in lists[:min(units, n_gw + n_gx)]]
    assert min(sizes) >= 1


def test_tile_plan_without_a_table_for_very_many_tiles():
    info, lists = lbp.lbp_test_tile_plan(3072, 768, 400, 16, 8, 74, 1, 1)
    assert not info["listed"] and lists is None


def test_binding_structs_have_the_size_the_library_was_compiled_with():
    # a field added to include/lbp.h and not to the ctypes declarations (or the
    # other way round) would shift every field behind it
    from paper_2309_15275_b200 import binding as B
    lib = B._lib()
    for which, cls in ((0, B.Layer), (1, B.Extras), (2, B.View), (3, B.Basis)):
        assert lib.lbp_test_struct_size(which) == ctypes.sizeof(cls), cls.__name__
    assert lib.lbp_test_struct_size(99) == 0
