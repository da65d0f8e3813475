"""Pins for the fp64 oracle: each test ties one part of oracle/lbp_oracle.py to
something fixed by the paper or by mathematics, not to the oracle itself.

A dropped term, wrong sign, transposed operand, wrong scale or wrong ordering
anywhere in the oracle should fail at least one of these.
"""
import os

import numpy as np
import pytest

from oracle import lbp_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
KS = (4, 8, 16)


def _read_kv(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = line.split()
            out[key] = float(val)
    return out


# ---------------------------------------------------------------- bases ----
@pytest.mark.parametrize("k", KS)
def test_hadamard_orthogonal_pm1(k):
    # "bases are orthogonal", "contain only +1 and -1" (Sec. 3)
    h = O.hadamard(k)
    assert set(np.unique(h)) == {-1, 1}
    assert np.array_equal(h @ h.T, k * np.eye(k, dtype=np.int64))
    assert np.array_equal(h, h.T)


def test_hadamard_order2_and_kron():
    # textbook: H_2 = [[1,1],[1,-1]], H_2k = H_2 (x) H_k
    h2 = np.array([[1, 1], [1, -1]])
    assert np.array_equal(O.hadamard(2), h2)
    for k in (2, 4, 8):
        assert np.array_equal(O.hadamard(2 * k), np.kron(h2, O.hadamard(k)))


def test_walsh_order4_rows():
    # the four sequency-ordered Walsh functions of length 4 (textbook)
    want = np.array([[1, 1, 1, 1], [1, 1, -1, -1], [1, -1, -1, 1], [1, -1, 1, -1]])
    assert np.array_equal(O.walsh(4), want)


def _bitrev(v, bits):
    r = 0
    for _ in range(bits):
        r = (r << 1) | (v & 1)
        v >>= 1
    return r


@pytest.mark.parametrize("k", KS)
def test_walsh_sequency_and_closed_form(k):
    wal = O.walsh(k)
    bits = k.bit_length() - 1
    h = O.hadamard(k)
    for s in range(k):
        assert O.sign_changes(wal[s]) == s
        # closed form: sequency s <-> Sylvester row bitreverse(gray(s))
        assert np.array_equal(wal[s], h[_bitrev(s ^ (s >> 1), bits)])
    assert np.array_equal(wal @ wal.T, k * np.eye(k, dtype=np.int64))


@pytest.mark.parametrize("k", KS)
def test_walsh_low_rows_are_run_constant(k):
    # a row with s < k/2^t sign changes whose runs are aligned is constant on
    # runs of 2^t: checks the ordering really is by frequency
    wal = O.walsh(k)
    t = 1
    while (k >> t) >= 1:
        run = 1 << t
        for s in range(k >> t):
            blocks = wal[s].reshape(-1, run)
            assert np.all(blocks == blocks[:, :1])
        t += 1


@pytest.mark.parametrize("k", KS)
def test_basis_flat_is_raster_outer_product(k):
    wal = O.walsh(k)
    for i, j in [(0, 0), (1, 0), (0, 1), (k - 1, 2), (3, k - 1)]:
        b = O.basis_flat(k, i, j)
        assert b.shape == (k * k,)
        for u, v in [(0, 0), (1, 2), (k - 1, 0), (2, k - 1), (k - 1, k - 1)]:
            assert b[u * k + v] == wal[i][u] * wal[j][v]
    # i indexes the H (row) axis: B_{1,0} changes sign along u, not along v
    b10 = O.basis_2d(k, 1, 0)
    assert np.all(b10 == b10[:, :1]) and b10[0, 0] == 1 and b10[k - 1, 0] == -1


@pytest.mark.parametrize("k", KS)
def test_bases_complete_and_orthogonal(k):
    # "complete" + "orthogonal": all k^2 flattened bases form k * orthogonal matrix
    allb = O.basis_matrix(k, [(i, j) for i in range(k) for j in range(k)])
    assert set(np.unique(allb)) == {-1, 1}
    assert np.array_equal(allb.T @ allb, k * k * np.eye(k * k, dtype=np.int64))


# ------------------------------------------------------------ selection ----
def test_selection_ranks_printed_in_paper():
    rule_id = {"L1": O.RULE_L1, "LINF": O.RULE_LINF}
    n = 0
    with open(os.path.join(GOLDEN, "lp_ranks.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rule, m, r = line.split()
            sel = O.select_bases(8, rule_id[rule], int(m))
            assert len(sel) == int(r), (rule, m)
            n += 1
    assert n == 6


@pytest.mark.parametrize("k", KS)
def test_selection_sets_by_definition(k):
    for m in range(1, k + 1):
        l1 = O.select_bases(k, O.RULE_L1, m)
        assert set(l1) == {(i, j) for i in range(k) for j in range(k) if i + j <= m - 1}
        assert len(l1) == m * (m + 1) // 2
        li = O.select_bases(k, O.RULE_LINF, m)
        assert set(li) == {(i, j) for i in range(k) for j in range(k) if max(i, j) <= m - 1}
        assert len(li) == m * m
        # prefix at a triangular rank is exactly the LP_L1 set, in the same order
        assert O.select_bases(k, O.RULE_PREFIX, m * (m + 1) // 2) == l1
    full = O.select_bases(k, O.RULE_PREFIX, k * k)
    assert sorted(full) == [(i, j) for i in range(k) for j in range(k)]
    for r in range(1, k * k):
        assert O.select_bases(k, O.RULE_PREFIX, r) == full[:r]        # nested


def test_prefix_order_listed_cases():
    assert O.select_bases(8, O.RULE_PREFIX, 2) == [(0, 0), (0, 1)]
    assert set(O.select_bases(8, O.RULE_PREFIX, 4)) == {(0, 0), (0, 1), (1, 0), (1, 1)}
    r8 = O.select_bases(8, O.RULE_PREFIX, 8)
    assert set(r8) == {(i, j) for i in range(3) for j in range(3) if i + j <= 2} | {(1, 2), (2, 1)}
    r16 = O.select_bases(8, O.RULE_PREFIX, 16)
    assert set(r16) == {(i, j) for i in range(8) for j in range(8) if i + j <= 4} | {(2, 3)}
    # DC basis is always first
    for k in KS:
        assert O.select_bases(k, O.RULE_PREFIX, 1) == [(0, 0)]


def test_selection_rejects_bad_arguments():
    with pytest.raises(ValueError):
        O.select_bases(8, O.RULE_PREFIX, 0)
    with pytest.raises(ValueError):
        O.select_bases(8, O.RULE_PREFIX, 65)
    with pytest.raises(ValueError):
        O.select_bases(8, O.RULE_LINF, 9)
    with pytest.raises(ValueError):
        O.project(np.zeros((1, 8, 8, 1)), 8, [(0, 0), (0, 0)])
    with pytest.raises(ValueError):
        O.project(np.zeros((1, 8, 8, 1)), 8, [(0, 8)])
    with pytest.raises(ValueError):
        O.project(np.zeros((1, 8, 12, 1)), 8, [(0, 0)])


# --------------------------------------------------- projection / expand ----
def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


@pytest.mark.parametrize("k", KS)
def test_projection_matches_pointwise_definition(k):
    # Eq. 6 written out as scalar loops on a tiny ragged-looking case
    B, Hb, Wb, C = 2, 2, 3, 3
    t = _rand((B, Hb * k, Wb * k, C), 1)
    bases = [(0, 0), (1, 0), (0, 2), (k - 1, k - 2), (2, 1)]
    wal = O.walsh(k)
    got = O.project(t, k, bases)
    assert got.shape == (B, Hb, Wb, len(bases), C)
    rng = np.random.default_rng(5)
    for _ in range(40):
        b, bh, bw = rng.integers(B), rng.integers(Hb), rng.integers(Wb)
        q, c = rng.integers(len(bases)), rng.integers(C)
        i, j = bases[q]
        acc = 0.0
        for u in range(k):
            for v in range(k):
                acc += wal[i][u] * wal[j][v] * t[b, bh * k + u, bw * k + v, c]
        assert got[b, bh, bw, q, c] == pytest.approx(acc / k, rel=1e-12, abs=1e-12)


@pytest.mark.parametrize("k", KS)
def test_expand_matches_pointwise_definition(k):
    B, Hb, Wb, C = 1, 2, 2, 2
    bases = [(0, 0), (0, 1), (1, 0), (3, 2)]
    th = _rand((B, Hb, Wb, len(bases), C), 2)
    wal = O.walsh(k)
    got = O.expand(th, k, bases)
    assert got.shape == (B, Hb * k, Wb * k, C)
    rng = np.random.default_rng(6)
    for _ in range(40):
        h, w, c = rng.integers(Hb * k), rng.integers(Wb * k), rng.integers(C)
        acc = sum(wal[i][h % k] * wal[j][w % k] * th[0, h // k, w // k, q, c]
                  for q, (i, j) in enumerate(bases))
        assert got[0, h, w, c] == pytest.approx(acc / k, rel=1e-12, abs=1e-12)


@pytest.mark.parametrize("k", KS)
def test_orthonormal_projector_properties(k):
    # P^T P = I_r ; project(expand(.)) = id ; Parseval at full rank,
    # contraction otherwise (Sec. 3.2: "WHT preserves the signal energy")
    t = _rand((2, 2 * k, k, 5), 3)
    for r in (1, 3, k, k * k // 2, k * k):
        bases = O.select_bases(k, O.RULE_PREFIX, r)
        P = O.basis_matrix(k, bases) / k
        assert np.allclose(P.T @ P, np.eye(r), atol=1e-14)
        th = O.project(t, k, bases)
        assert np.allclose(O.project(O.expand(th, k, bases), k, bases), th, atol=1e-12)
        e_in, e_hat = np.sum(t * t), np.sum(th * th)
        if r == k * k:
            assert e_hat == pytest.approx(e_in, rel=1e-12)
            assert np.allclose(O.expand(th, k, bases), t, atol=1e-12)   # lossless
        else:
            assert e_hat < e_in


def test_blocks_are_origin_aligned_and_non_overlapping():
    # a delta at (h, w) must only excite the block that contains it
    k = 4
    t = np.zeros((1, 8, 12, 1))
    t[0, 5, 9, 0] = 1.0
    th = O.project(t, k, O.select_bases(k, O.RULE_PREFIX, 16))
    nz = np.argwhere(np.abs(th).sum(axis=(3, 4)) > 0)
    assert nz.tolist() == [[0, 1, 2]]
    back = O.expand(th, k, O.select_bases(k, O.RULE_PREFIX, 16))
    assert np.allclose(back, t, atol=1e-14)


def test_r1_is_average_pool_times_k():
    # DC coefficient = (1/k) * sum over the block = k * mean (textbook)
    k = 8
    t = _rand((2, 16, 8, 3), 4)
    th = O.project(t, k, [(0, 0)])
    pooled = t.reshape(2, 2, k, 1, k, 3).mean(axis=(2, 4))
    assert np.allclose(th[:, :, :, 0, :], k * pooled, atol=1e-12)
    up = O.expand(th, k, [(0, 0)])
    want = np.repeat(np.repeat(pooled, k, axis=1), k, axis=2)
    assert np.allclose(up, want, atol=1e-12)


# ------------------------------------------------------------- backward ----
def _tiny(k, seed, B=2, Hb=2, Wb=1, Cin=5, Cout=4):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, Hb * k, Wb * k, Cin))
    gy = rng.standard_normal((B, Hb * k, Wb * k, Cout))
    w = rng.standard_normal((Cout, Cin))
    return x, gy, w


def test_exact_bp_matches_finite_differences():
    # Eq. 2 pinned to calculus: loss = <y, g_y>, y = x w^T
    x, gy, w = _tiny(4, 7, B=1, Hb=1, Wb=1, Cin=3, Cout=2)
    gx, gw = O.backward_exact(x, gy, w)
    assert gx.shape == x.shape and gw.shape == w.shape

    def loss(xx, ww):
        return float(np.sum((xx.reshape(-1, 3) @ ww.T) * gy.reshape(-1, 2)))

    eps = 1e-6
    for idx in [(0, 0, 0, 0), (0, 3, 2, 1), (0, 1, 3, 2)]:
        xp = x.copy(); xp[idx] += eps
        xm = x.copy(); xm[idx] -= eps
        assert gx[idx] == pytest.approx((loss(xp, w) - loss(xm, w)) / (2 * eps), rel=1e-6)
    for idx in [(0, 0), (1, 2), (0, 1)]:
        wp = w.copy(); wp[idx] += eps
        wm = w.copy(); wm[idx] -= eps
        assert gw[idx] == pytest.approx((loss(x, wp) - loss(x, wm)) / (2 * eps), rel=1e-6)


@pytest.mark.parametrize("k", KS)
def test_full_rank_reproduces_exact_bp(k):
    # "lossless when all bases are activated" (Sec. 3)
    x, gy, w = _tiny(k, 8)
    bases = O.select_bases(k, O.RULE_PREFIX, k * k)
    gx, gw = O.backward_lowrank(x, gy, w, k, bases)
    ex, ew = O.backward_exact(x, gy, w)
    assert np.allclose(gx, ex, rtol=1e-12, atol=1e-12)
    assert np.allclose(gw, ew, rtol=1e-12, atol=1e-12)
    # any permutation of the full set gives the same gradients
    perm = list(reversed(bases))
    gx2, gw2 = O.backward_lowrank(x, gy, w, k, perm)
    assert np.allclose(gx2, ex, atol=1e-12) and np.allclose(gw2, ew, atol=1e-12)


@pytest.mark.parametrize("k,r", [(4, 3), (4, 7), (8, 8), (8, 21), (16, 10)])
def test_low_rank_equals_dense_projector_route(k, r):
    # brute force: Pi = P P^T (k^2 x k^2) applied per block to exact quantities
    x, gy, w = _tiny(k, 9 + r)
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    gx, gw = O.backward_lowrank(x, gy, w, k, bases)

    wal = O.walsh(k)
    Pi = np.zeros((k * k, k * k))
    for (i, j) in bases:                       # built without basis_matrix()
        b = np.array([wal[i][u] * wal[j][v] for u in range(k) for v in range(k)], float)
        Pi += np.outer(b, b) / (k * k)
    assert np.allclose(Pi @ Pi, Pi, atol=1e-13) and np.allclose(Pi, Pi.T)

    def apply_pi(t):
        B, H, W_, C = t.shape
        out = np.zeros_like(t)
        for b in range(B):
            for bh in range(H // k):
                for bw in range(W_ // k):
                    blk = t[b, bh * k:(bh + 1) * k, bw * k:(bw + 1) * k, :].reshape(k * k, C)
                    out[b, bh * k:(bh + 1) * k, bw * k:(bw + 1) * k, :] = (Pi @ blk).reshape(k, k, C)
        return out

    Cin, Cout = x.shape[-1], gy.shape[-1]
    exact_gx = (gy.reshape(-1, Cout) @ w).reshape(x.shape)
    assert np.allclose(gx, apply_pi(exact_gx), atol=1e-12)            # Pi (g_y w)
    assert np.allclose(gx, (apply_pi(gy).reshape(-1, Cout) @ w).reshape(x.shape), atol=1e-12)
    gw_a = apply_pi(gy).reshape(-1, Cout).T @ x.reshape(-1, Cin)      # (Pi g_y)^T x
    gw_b = gy.reshape(-1, Cout).T @ apply_pi(x).reshape(-1, Cin)      # g_y^T (Pi x)
    assert np.allclose(gw, gw_a, atol=1e-11) and np.allclose(gw, gw_b, atol=1e-11)


def test_r1_backward_is_pooled_bp():
    k = 8
    x, gy, w = _tiny(k, 21, B=2, Hb=1, Wb=2, Cin=3, Cout=4)
    gx, gw = O.backward_lowrank(x, gy, w, k, [(0, 0)])
    px = x.reshape(2, 1, k, 2, k, 3).mean(axis=(2, 4)).reshape(-1, 3)
    pg = gy.reshape(2, 1, k, 2, k, 4).mean(axis=(2, 4)).reshape(-1, 4)
    assert np.allclose(gw, k * k * pg.T @ px, atol=1e-12)
    want = np.repeat(np.repeat((pg @ w).reshape(2, 1, 2, 3), k, axis=1), k, axis=2)
    assert np.allclose(gx, want, atol=1e-12)


def test_block_constant_inputs_are_exact_at_r1():
    k = 4
    rng = np.random.default_rng(22)
    xc = np.repeat(np.repeat(rng.standard_normal((2, 2, 3, 5)), k, axis=1), k, axis=2)
    gc = np.repeat(np.repeat(rng.standard_normal((2, 2, 3, 6)), k, axis=1), k, axis=2)
    w = rng.standard_normal((6, 5))
    gx, gw = O.backward_lowrank(xc, gc, w, k, [(0, 0)])
    ex, ew = O.backward_exact(xc, gc, w)
    assert np.allclose(gx, ex, atol=1e-12) and np.allclose(gw, ew, atol=1e-12)


@pytest.mark.parametrize("k,r", [(4, 5), (8, 8), (8, 36), (16, 3)])
def test_outputs_are_coupled_through_w(k, r):
    # <g_x~, x> = <g_w~, w> for every basis set (both equal <g_y_hat, x_hat w^T>)
    x, gy, w = _tiny(k, 30 + r)
    gx, gw = O.backward_lowrank(x, gy, w, k, O.select_bases(k, O.RULE_PREFIX, r))
    assert np.sum(gx * x) == pytest.approx(np.sum(gw * w), rel=1e-10)


def test_basis_order_changes_only_t_hat_axis():
    k = 8
    x, gy, w = _tiny(k, 40)
    bases = O.select_bases(k, O.RULE_L1, 3)
    perm = [bases[i] for i in (3, 0, 5, 1, 4, 2)]
    a = O.backward_lowrank(x, gy, w, k, bases)
    b = O.backward_lowrank(x, gy, w, k, perm)
    assert np.allclose(a[0], b[0], atol=1e-12) and np.allclose(a[1], b[1], atol=1e-12)
    th, thp = O.project(x, k, bases), O.project(x, k, perm)
    assert np.allclose(thp, th[:, :, :, (3, 0, 5, 1, 4, 2), :], atol=0)


def test_batch_and_blocks_sum_into_gw():
    # g_W over a batch = sum of per-image g_W; g_x of image b depends on image b only
    k = 4
    x, gy, w = _tiny(k, 41, B=3)
    bases = O.select_bases(k, O.RULE_PREFIX, 6)
    gx, gw = O.backward_lowrank(x, gy, w, k, bases)
    acc = np.zeros_like(gw)
    for b in range(3):
        gxb, gwb = O.backward_lowrank(x[b:b + 1], gy[b:b + 1], w, k, bases)
        acc += gwb
        assert np.allclose(gxb[0], gx[b], atol=1e-13)
    assert np.allclose(acc, gw, atol=1e-12)


# ----------------------------------------------------------- cost model ----
def test_flops_worked_example_from_paper():
    g = _read_kv(os.path.join(GOLDEN, "flops_worked_example.txt"))
    f = O.flops(int(g["Cx"]), int(g["Cy"]), int(g["L"]), int(g["r"]))
    mf = {n: v / 1e6 for n, v in f.items()}
    lbp = mf["projection"] + mf["lowrank_mm"] + mf["reverse_projection"]
    over = mf["projection"] + mf["reverse_projection"]
    tol = 0.1 + 1e-9                       # printed to one decimal
    # 4*3072*768*49 = 462.42 M; the paper prints 462.3 (0.03 % low), so the
    # vanilla figure alone gets 0.15 MFLOPs of slack
    assert abs(mf["vanilla"] - g["vanilla_mflops"]) <= 0.15
    assert abs(lbp - g["lbp_total_mflops"]) <= tol
    assert abs(mf["projection"] - g["projection_mflops"]) <= tol
    assert abs(mf["lowrank_mm"] - g["lowrank_mm_mflops"]) <= tol
    assert abs(mf["reverse_projection"] - g["reverse_projection_mflops"]) <= tol
    assert abs(over - g["overhead_mflops"]) <= tol
    assert abs(100 * lbp / mf["vanilla"] - g["lbp_over_vanilla_percent"]) <= tol
    assert abs(100 * over / mf["vanilla"] - g["overhead_over_vanilla_percent"]) <= tol
    assert abs(100 * over / lbp - g["overhead_over_lbp_percent"]) <= tol
    # overhead ratio of Sec. 3.3: (2Cx+Cy) L r / (4 Cx Cy L), which simplifies to
    # (1/Cy + 1/(2Cx)) r/2 (the paper's simplified form has Cx and Cy swapped)
    cx, cy, L, r = g["Cx"], g["Cy"], g["L"], g["r"]
    assert over / mf["vanilla"] == pytest.approx((2 * cx + cy) * L * r / (4 * cx * cy * L), rel=1e-12)
    assert over / mf["vanilla"] == pytest.approx((1 / cy + 1 / (2 * cx)) * r / 2, rel=1e-12)


# ------------------------------------------- LHE selection (Sec. 3.2) ----
@pytest.mark.parametrize("k", KS)
def test_spectrum_preserves_energy(k):
    # Parseval (Sec. 3.2): the orthonormal WHT keeps the signal energy, so the
    # energies of all k^2 responses add up to ||t||^2.
    rng = np.random.default_rng(5)
    t = rng.standard_normal((2, 2 * k, k, 3))
    E = O.spectrum(t, k)
    assert E.shape == (k, k) and np.all(E >= 0)
    assert abs(E.sum() - np.sum(t * t)) <= 1e-10 * np.sum(t * t)


@pytest.mark.parametrize("k", KS)
def test_spectrum_matches_pointwise_definition(k):
    # brute force from the definition of a response: Python loops over the
    # block, Walsh rows built here from their sign-change count
    rng = np.random.default_rng(6)
    t = rng.standard_normal((1, k, 2 * k, 2))
    H = np.array([[(-1) ** bin(a & b).count("1") for b in range(k)] for a in range(k)])
    wal = {int(np.sum(H[a, 1:] != H[a, :-1])): H[a] for a in range(k)}
    E = np.zeros((k, k))
    for bw in range(2):
        for c in range(2):
            for i in range(k):
                for j in range(k):
                    acc = 0.0
                    for u in range(k):
                        for v in range(k):
                            acc += wal[i][u] * wal[j][v] * t[0, u, bw * k + v, c]
                    E[i, j] += (acc / k) ** 2
    assert np.allclose(O.spectrum(t, k), E, rtol=1e-12, atol=1e-12)


def test_spectrum_of_a_single_basis_function_is_a_single_peak():
    # a block equal to amplitude * B_{i,j} has all its energy in response (i, j):
    # pins the index order (i along H, j along W) and the orientation
    k, i, j = 8, 2, 5
    amp = np.array([1.0, -3.0, 0.5])
    blk = O.basis_2d(k, i, j).astype(np.float64)                  # k x k, rows = H axis
    t = (blk[None, :, :, None] * amp[None, None, None, :])
    E = O.spectrum(t, k)
    expect = np.zeros((k, k))
    expect[i, j] = k * k * np.sum(amp ** 2)                       # ||t||^2
    assert np.allclose(E, expect, atol=1e-9)
    # the transposed pattern peaks at (j, i)
    E2 = O.spectrum(np.transpose(t, (0, 2, 1, 3)), k)
    assert np.argmax(E2) == j * k + i


def test_block_constant_tensor_has_only_dc_energy():
    k = 4
    rng = np.random.default_rng(8)
    coarse = rng.standard_normal((2, 3, 2, 5))
    t = np.repeat(np.repeat(coarse, k, axis=1), k, axis=2)
    E = O.spectrum(t, k)
    assert E[0, 0] > 0 and np.allclose(np.delete(E.ravel(), 0), 0.0, atol=1e-12)


def test_lhe_selection_takes_the_strongest_and_breaks_ties_by_frequency():
    k = 4
    E = np.zeros((k, k))
    E[3, 3], E[0, 2], E[2, 0], E[1, 1], E[0, 0] = 9.0, 5.0, 5.0, 5.0, 1.0
    # three equal energies on the anti-diagonal i + j = 2: the balanced pair
    # first, then the smaller row index (the PREFIX order key)
    assert O.select_lhe(E, k, 5) == [(3, 3), (1, 1), (0, 2), (2, 0), (0, 0)]
    assert O.select_lhe(E, k, 1) == [(3, 3)]
    full = O.select_lhe(E, k, k * k)
    assert sorted(full) == [(i, j) for i in range(k) for j in range(k)]
    with pytest.raises(ValueError):
        O.select_lhe(E, k, 0)


def test_lhe_on_a_decaying_spectrum_equals_the_low_pass_set():
    # energy that falls strictly with the PREFIX order key: the strongest r
    # responses are exactly the PREFIX-r (for triangular r: LP_L1) set
    k = 8
    order = O.select_bases(k, O.RULE_PREFIX, k * k)
    E = np.zeros((k, k))
    for rank, (i, j) in enumerate(order):
        E[i, j] = 2.0 ** (-rank)
    for r in (1, 3, 8, 10, 21):
        assert O.select_lhe(E, k, r) == order[:r]
    assert set(O.select_lhe(E, k, 10)) == set(O.select_bases(k, O.RULE_L1, 4))


# ------------------------------------------------------- error measures ----
def test_rel_fro_is_the_relative_frobenius_error():
    # every parity assertion goes through these: pin them to hand-computed values
    b = np.array([[3.0, 4.0], [0.0, 12.0]])                      # ||b|| = 13
    assert O.rel_fro(b * (1 + 1e-3), b) == pytest.approx(1e-3, rel=1e-12)
    assert O.rel_fro(b + np.array([[0.0, 0.0], [5.0, 0.0]]), b) == pytest.approx(5.0 / 13.0, rel=1e-12)
    assert O.rel_fro(np.array([1.0, 0.0]), np.array([0.0, 1.0])) == pytest.approx(np.sqrt(2.0))
    assert O.rel_fro(b, b) == 0.0
    # the reference is the second argument (the denominator)
    assert O.rel_fro(2 * b, b) == pytest.approx(1.0) and O.rel_fro(b, 2 * b) == pytest.approx(0.5)
    # zero reference: the absolute error
    assert O.rel_fro(np.array([3.0, 4.0]), np.zeros(2)) == pytest.approx(5.0)


def test_local_error_measures_find_one_bad_patch():
    k = 4
    rng = np.random.default_rng(21)
    ref = rng.standard_normal((2, 2 * k, 3 * k, 5))
    got = ref.copy()
    got[1, k:2 * k, 2 * k:3 * k, :] *= 1.5                        # one block off by 50 %
    assert O.block_rel_fro(got, ref, k) == pytest.approx(0.5, rel=1e-12)
    assert O.rel_fro(got, ref) < 0.25                             # diluted in the global norm
    assert O.block_rel_fro(ref, ref, k) == 0.0
    m = rng.standard_normal((300, 200))
    bad = m.copy()
    bad[256:300, 128:200] *= 3.0                                  # the ragged corner tile
    assert O.tile_rel_fro(bad, m, 128) == pytest.approx(2.0, rel=1e-12)
    assert O.rel_fro(bad, m) < 1.0
    bad2 = m.copy()
    bad2[0, 0] += 1.0
    t00 = np.linalg.norm(m[:128, :128])
    assert O.tile_rel_fro(bad2, m, 128) == pytest.approx(1.0 / t00, rel=1e-12)


# ------------------------------------- x_hat handed in (Eq. 3, Alg. 1) ----
@pytest.mark.parametrize("k,r", [(4, 5), (8, 8), (16, 3)])
def test_projected_backward_is_vanilla_bp_on_the_expanded_coefficients(k, r):
    # g_w = g_y_hat^T x_hat = (P^T g_y)^T x_hat = g_y^T (P x_hat): Eq. 2 with x
    # replaced by p^{-1}(x_hat), for ANY coefficient tensor (not only projections)
    rng = np.random.default_rng(31 + k)
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    B, Hb, Wb, Cin, Cout = 2, 2, 1, 5, 4
    x_hat = rng.standard_normal((B, Hb, Wb, r, Cin))
    gy = rng.standard_normal((B, Hb * k, Wb * k, Cout))
    w = rng.standard_normal((Cout, Cin))
    gx, gw = O.backward_lowrank_projected(x_hat, gy, w, k, bases)
    _, gw_ref = O.backward_exact(O.expand(x_hat, k, bases), gy, w)
    assert np.allclose(gw, gw_ref, rtol=1e-12, atol=1e-12)
    # g_x does not depend on x_hat: the dense projector applied to g_y w
    P = O.basis_matrix(k, bases).astype(np.float64) / k
    Pi = P @ P.T
    exact_gx = O.to_blocks((gy.reshape(-1, Cout) @ w).reshape(B, Hb * k, Wb * k, Cin), k)
    want = O.from_blocks(np.einsum("pq,bhwqc->bhwpc", Pi, exact_gx), k)
    assert np.allclose(gx, want, rtol=1e-12, atol=1e-12)


def test_projected_backward_equals_algorithm_1_when_x_hat_is_p_of_x():
    k, r = 8, 10
    x, gy, w = _tiny(k, 41)
    bases = O.select_bases(k, O.RULE_PREFIX, r)
    a = O.backward_lowrank(x, gy, w, k, bases)
    b = O.backward_lowrank_projected(O.project(x, k, bases), gy, w, k, bases)
    assert np.allclose(a[0], b[0], atol=1e-13) and np.allclose(a[1], b[1], atol=1e-12)
    with pytest.raises(ValueError):
        O.backward_lowrank_projected(O.project(x, k, bases)[:, :1], gy, w, k, bases)


# ------------------------------------ grids that are not multiples of k ----
def test_padding_goes_to_the_high_end_of_the_grid():
    # a single token at the last real position (6, 6) of a 7 x 7 map, order 8:
    # its coefficients are wal_i[6] wal_j[6] / 8 -- it sits at (6, 6) of the block,
    # so the zero tokens were appended after it, not before
    k = 8
    t = np.zeros((1, 7, 7, 1))
    t[0, 6, 6, 0] = 2.0
    pairs = [(i, j) for i in range(k) for j in range(k)]
    th = O.project_padded(t, k, pairs)
    assert th.shape == (1, 1, 1, 64, 1)
    wal = O.walsh(k)
    want = np.array([wal[i][6] * wal[j][6] * 2.0 / k for (i, j) in pairs])
    assert np.allclose(th[0, 0, 0, :, 0], want, atol=1e-15)
    assert O.pad_grid(t, k).shape == (1, 8, 8, 1) and O.pad_grid(t, k)[0, 7, 7, 0] == 0.0
    assert O.pad_grid(np.ones((1, 8, 16, 2)), 8).shape == (1, 8, 16, 2)


@pytest.mark.parametrize("k,H,W", [(8, 7, 7), (4, 7, 7), (8, 14, 14), (4, 6, 9)])
def test_padded_full_rank_is_exact_bp_on_the_real_tokens(k, H, W):
    rng = np.random.default_rng(50 + k + H)
    x = rng.standard_normal((2, H, W, 6))
    gy = rng.standard_normal((2, H, W, 3))
    w = rng.standard_normal((3, 6))
    pairs = O.select_bases(k, O.RULE_PREFIX, k * k)
    gx, gw = O.backward_lowrank_padded(x, gy, w, k, pairs)
    ex, ew = O.backward_exact(x, gy, w)
    assert gx.shape == x.shape
    assert np.allclose(gx, ex, atol=1e-12) and np.allclose(gw, ew, atol=1e-11)


def test_padded_rank1_pools_over_the_real_tokens_of_a_block():
    # r = 1 (DC only): every real token of a block receives
    # (sum of g_y over the block's real tokens / k^2) w, partial blocks included
    k, H, W = 4, 6, 7
    rng = np.random.default_rng(61)
    x = rng.standard_normal((1, H, W, 3))
    gy = rng.standard_normal((1, H, W, 2))
    w = rng.standard_normal((2, 3))
    gx, gw = O.backward_lowrank_padded(x, gy, w, k, [(0, 0)])
    want_w = np.zeros((2, 3))
    for bh in range(2):
        for bw in range(2):
            hs, ws_ = slice(bh * k, min(H, bh * k + k)), slice(bw * k, min(W, bw * k + k))
            sg = gy[0, hs, ws_].reshape(-1, 2).sum(axis=0)
            sx = x[0, hs, ws_].reshape(-1, 3).sum(axis=0)
            assert np.allclose(gx[0, hs, ws_], (sg / (k * k)) @ w, atol=1e-13)
            want_w += np.outer(sg, sx) / (k * k)
    assert np.allclose(gw, want_w, atol=1e-12)


def test_padded_equals_plain_on_divisible_grids():
    k = 8
    x, gy, w = _tiny(k, 71)
    bases = O.select_bases(k, O.RULE_L1, 3)
    a = O.backward_lowrank(x, gy, w, k, bases)
    b = O.backward_lowrank_padded(x, gy, w, k, bases)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# ------------------------- tokens outside the grid, bias, accumulation ----
def test_class_token_rows_take_vanilla_bp_and_complete_the_layer():
    # a (B, 1 + H W, C) ViT tensor: grid tokens at full rank plus the class token
    # by Eq. 2 must add up to vanilla BP over all 1 + H W tokens
    k, B, Cin, Cout = 4, 3, 5, 4
    rng = np.random.default_rng(81)
    xt = rng.standard_normal((B, 1 + k * k, Cin))
    gt = rng.standard_normal((B, 1 + k * k, Cout))
    w = rng.standard_normal((Cout, Cin))
    pairs = O.select_bases(k, O.RULE_PREFIX, k * k)
    gx_grid, gw_grid = O.backward_lowrank(xt[:, 1:].reshape(B, k, k, Cin),
                                          gt[:, 1:].reshape(B, k, k, Cout), w, k, pairs)
    gx_cls, gw_cls = O.backward_extra_tokens(xt[:, 0], gt[:, 0], w)
    ex, ew = O.backward_exact(xt, gt, w)
    assert np.allclose(gw_grid + gw_cls, ew, atol=1e-11)
    assert np.allclose(gx_cls, ex[:, 0], atol=1e-12)
    assert np.allclose(gx_grid.reshape(B, k * k, Cin), ex[:, 1:], atol=1e-12)
    # orientation: one token, one non-zero entry each
    gxe, gwe = O.backward_extra_tokens(np.eye(1, Cin, 2), np.eye(1, Cout, 1) * 3.0, w)
    assert gwe[1, 2] == 3.0 and np.count_nonzero(gwe) == 1
    assert np.allclose(gxe[0], 3.0 * w[1])


def test_bias_gradient_is_the_token_sum_and_k_times_the_dc_coefficients():
    k = 8
    rng = np.random.default_rng(91)
    gy = rng.standard_normal((2, 2 * k, k, 5))
    cls = rng.standard_normal((2, 5))
    # finite differences of L = <g_y, y + bias> in the bias: dL/db_c = sum of g_y[..., c]
    want = np.array([gy[..., c].sum() for c in range(5)])
    assert np.allclose(O.bias_grad(gy), want, atol=1e-12)
    assert np.allclose(O.bias_grad(gy, cls), want + cls.sum(axis=0), atol=1e-12)
    # closed form through Eq. 6: B_{0,0} is all ones, so the (0,0) coefficient of a
    # block is (sum of its tokens) / k
    for bases in ([(0, 0)], O.select_bases(k, O.RULE_L1, 3)):
        q = bases.index((0, 0))
        dc = O.project(gy, k, bases)[:, :, :, q, :]
        assert np.allclose(k * dc.sum(axis=(0, 1, 2)), want, atol=1e-12)
    # holds on a zero-extended grid too (the zero tokens add nothing)
    g7 = rng.standard_normal((1, 7, 7, 3))
    dc7 = O.project_padded(g7, k, [(0, 0)])[:, :, :, 0, :]
    assert np.allclose(k * dc7.sum(axis=(0, 1, 2)), O.bias_grad(g7), atol=1e-12)


def test_accumulation_over_micro_batches_equals_one_big_batch():
    k = 4
    x, gy, w = _tiny(k, 95, B=4)
    bases = O.select_bases(k, O.RULE_L1, 2)
    _, whole = O.backward_lowrank(x, gy, w, k, bases)
    _, first = O.backward_lowrank(x[:2], gy[:2], w, k, bases)
    _, second = O.backward_lowrank(x[2:], gy[2:], w, k, bases)
    assert np.allclose(O.accumulate(second, first, 1.0), whole, atol=1e-12)
    assert np.array_equal(O.accumulate(second, first, 0.0), second)
    assert np.array_equal(O.accumulate(second), second)
