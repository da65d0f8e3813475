"""fp64 CPU oracle for LBP-WHT linear-layer backward.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the path computes, written from
the paper's definitions.  It is used by the tests, by the smoke check and by
the benchmark's CPU-baseline leg, and by nothing else: the product path never
imports it and it imports nothing from the product path.

Everything is numpy in float64.  No blocking, fusion, fast transform or
reordering beyond what the cited definition states; `numpy.matmul` /
`numpy.einsum` stand in for "matrix multiplication" where the paper writes one.

Readings of the paper taken here (the paper is silent or inconsistent):
  * token-major orientation: x is (tokens, Cx); g_w = g_y^T x; g_x = g_y w
    (Eq. 2 and Algorithm 1 read so that the shapes agree with w in R^{Cy x Cx});
  * the bases are scaled by 1/k in the projection and 1/k in the reverse
    projection, so that P^T P = I_r, signal energy is preserved (Sec. 3.2,
    Parseval) and the full-rank case reproduces exact backpropagation
    (Sec. 3, "lossless when all bases are activated");
  * basis index = sequency (number of sign changes of the Walsh row), the
    order in which a smaller index is a lower frequency (Sec. 3.2);
  * LP_L1-m is {(i,j): i+j <= m-1} with 0-based indices, which gives the rank
    m(m+1)/2 the tables print (Eq. 8 has an off-by-one as typeset);
  * the order-n transform is applied to non-overlapping k x k blocks of the
    (H, W) token grid; the batch and the blocks are just more blocks.

Parity status: every function below is pinned by tests/test_oracle_pins.py
(closed forms, invariants, a brute-force dense-projector route, textbook
special cases, the paper's printed ranks and FLOP figures), except
`lowrank error vs exact BP at r < k^2`, for which the paper gives no bound:
"parity unpinned" for that quantity only (it is not an output of the path).
The variants for real ViT token maps (zero-extended grids, tokens outside the
grid, bias gradient, accumulation, x_hat handed in) are pinned there too.
"""
from __future__ import annotations

import numpy as np

RULE_L1, RULE_LINF, RULE_PREFIX = 0, 1, 2


# --------------------------------------------------------------------------
# Bases (Sec. 3, Fig. 2c caption): order-n 2-D WHT bases B_{i,j}, +-1 entries
# --------------------------------------------------------------------------
def hadamard(k: int) -> np.ndarray:
    """Sylvester Hadamard matrix H_k[a, b] = (-1)^{popcount(a & b)}, k = 2^p."""
    if k < 1 or (k & (k - 1)) != 0:
        raise ValueError("order must be a power of two")
    h = np.empty((k, k), dtype=np.int64)
    for a in range(k):
        for b in range(k):
            h[a, b] = -1 if bin(a & b).count("1") & 1 else 1
    return h


def sign_changes(row: np.ndarray) -> int:
    return int(np.count_nonzero(row[1:] != row[:-1]))


def walsh(k: int) -> np.ndarray:
    """Walsh matrix: row s is the Hadamard row with exactly s sign changes.

    "Smaller index = lower frequency" (Sec. 3.2): frequency of a +-1 row is
    its number of sign changes, so the rows are ordered by counting them.
    """
    h = hadamard(k)
    wal = np.zeros((k, k), dtype=np.int64)
    seen = set()
    for a in range(k):
        s = sign_changes(h[a])
        if s in seen:
            raise AssertionError("two Hadamard rows with equal sequency")
        seen.add(s)
        wal[s] = h[a]
    if seen != set(range(k)):
        raise AssertionError("sequencies do not cover 0..k-1")
    return wal


def basis_2d(k: int, i: int, j: int) -> np.ndarray:
    """B_{i,j} as a k x k matrix: B[u, v] = wal_i[u] * wal_j[v] (i along H)."""
    wal = walsh(k)
    return np.outer(wal[i], wal[j])


def basis_flat(k: int, i: int, j: int) -> np.ndarray:
    """B_{i,j} flattened in raster order to length k^2 (Fig. 2c caption)."""
    return basis_2d(k, i, j).reshape(k * k)


# --------------------------------------------------------------------------
# Basis selection (Sec. 3.2, Eq. 8-9)
# --------------------------------------------------------------------------
def _prefix_key(i: int, j: int):
    # anti-diagonal first (L1 norm), then the more balanced pair, then row.
    return (i + j, max(i, j), i)


def select_bases(k: int, rule: int, param: int):
    """Ordered list of 0-based (i, j) pairs.

    RULE_L1,   param = m: {(i,j): i + j <= m-1}          r = m(m+1)/2 (m <= k)
    RULE_LINF, param = m: {(i,j): max(i,j) <= m-1}       r = m^2
    RULE_PREFIX, param = r: first r pairs of the total order
        key(i,j) = (i+j, max(i,j), i)  -- nests every LP_L1 set.
    All three are listed in that same total order.
    """
    pairs = [(i, j) for i in range(k) for j in range(k)]
    pairs.sort(key=lambda p: _prefix_key(*p))
    if rule == RULE_L1:
        if not 1 <= param <= 2 * k - 1:
            raise ValueError("LP_L1 parameter out of range")
        return [p for p in pairs if p[0] + p[1] <= param - 1]
    if rule == RULE_LINF:
        if not 1 <= param <= k:
            raise ValueError("LP_Linf parameter out of range")
        return [p for p in pairs if max(p) <= param - 1]
    if rule == RULE_PREFIX:
        if not 1 <= param <= k * k:
            raise ValueError("prefix rank out of range")
        return pairs[:param]
    raise ValueError("unknown rule")


def basis_matrix(k: int, bases) -> np.ndarray:
    """(B_{i1,j1} ... B_{ir,jr}) as a k^2 x r matrix of +-1 (Eq. 6)."""
    cols = [basis_flat(k, i, j) for (i, j) in bases]
    return np.stack(cols, axis=1).astype(np.int64)


def _check_bases(k: int, bases):
    if len(bases) < 1 or len(bases) > k * k:
        raise ValueError("rank out of range")
    if len(set(map(tuple, bases))) != len(bases):
        raise ValueError("duplicate basis")
    for (i, j) in bases:
        if not (0 <= i < k and 0 <= j < k):
            raise ValueError("basis index out of range")


# --------------------------------------------------------------------------
# Blocking of the token grid (reading: non-overlapping k x k blocks)
# --------------------------------------------------------------------------
def to_blocks(t: np.ndarray, k: int) -> np.ndarray:
    """(B,H,W,C) -> (B, H/k, W/k, k*k, C); position u*k+v inside a block."""
    B, H, W, C = t.shape
    if H % k or W % k:
        raise ValueError("grid not divisible by block size")
    t6 = t.reshape(B, H // k, k, W // k, k, C)          # b, bh, u, bw, v, c
    return t6.transpose(0, 1, 3, 2, 4, 5).reshape(B, H // k, W // k, k * k, C)


def from_blocks(tb: np.ndarray, k: int) -> np.ndarray:
    """Inverse of to_blocks."""
    B, Hb, Wb, kk, C = tb.shape
    t6 = tb.reshape(B, Hb, Wb, k, k, C).transpose(0, 1, 3, 2, 4, 5)
    return t6.reshape(B, Hb * k, Wb * k, C)


# --------------------------------------------------------------------------
# Projection / reverse projection (Eq. 6, Eq. 7)
# --------------------------------------------------------------------------
def project(t, k: int, bases) -> np.ndarray:
    """p(t) = t . (B_{i1,j1} ... B_{ir,jr}) / k, per block and channel.

    t (B,H,W,C) -> t_hat (B, H/k, W/k, r, C), q in the order of `bases`.
    """
    _check_bases(k, bases)
    t = np.asarray(t, dtype=np.float64)
    P = basis_matrix(k, bases).astype(np.float64) / k   # k^2 x r
    tb = to_blocks(t, k)                                # ..., k^2, C
    return np.einsum("pq,bhwpc->bhwqc", P, tb)


def expand(t_hat, k: int, bases) -> np.ndarray:
    """p^{-1}(t_hat) = t_hat . (B ...)^T / k.  (B,H/k,W/k,r,C) -> (B,H,W,C)."""
    _check_bases(k, bases)
    t_hat = np.asarray(t_hat, dtype=np.float64)
    P = basis_matrix(k, bases).astype(np.float64) / k
    tb = np.einsum("pq,bhwqc->bhwpc", P, t_hat)
    return from_blocks(tb, k)


# --------------------------------------------------------------------------
# Low-heuristic-error selection (Sec. 3.2): profile the energy of every basis
# response, keep the r strongest.
# --------------------------------------------------------------------------
def spectrum(t, k: int) -> np.ndarray:
    """E[i, j] = sum over blocks and channels of t_hat[.., (i,j), ..]^2 with all
    k^2 bases active (orthonormal coefficients, so sum(E) = ||t||^2 by Parseval).

    t (B,H,W,C) -> E (k, k), i the sequency along H, j along W.
    """
    all_pairs = [(i, j) for i in range(k) for j in range(k)]
    t_hat = project(t, k, all_pairs)                     # (B, H/k, W/k, k^2, C)
    return np.sum(t_hat * t_hat, axis=(0, 1, 2, 4)).reshape(k, k)


def select_lhe(energy, k: int, r: int):
    """The r bases with the largest energy, strongest first.  The paper does not
    say how equal energies are ordered; here the lower-frequency pair (the
    PREFIX order key) wins a tie, which makes the list unique."""
    energy = np.asarray(energy, dtype=np.float64).reshape(k, k)
    if not (1 <= r <= k * k):
        raise ValueError("rank out of range")
    pairs = [(i, j) for i in range(k) for j in range(k)]
    pairs.sort(key=lambda ij: (-energy[ij[0], ij[1]],) + _prefix_key(*ij))
    return pairs[:r]


# --------------------------------------------------------------------------
# Backward passes
# --------------------------------------------------------------------------
def backward_exact(x, g_y, w):
    """Vanilla BP (Eq. 2): g_w = g_y^T x over all tokens, g_x = g_y w."""
    x = np.asarray(x, dtype=np.float64)
    g_y = np.asarray(g_y, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    Cin, Cout = x.shape[-1], g_y.shape[-1]
    x2 = x.reshape(-1, Cin)
    g2 = g_y.reshape(-1, Cout)
    g_w = g2.T @ x2
    g_x = (g2 @ w).reshape(x.shape)
    return g_x, g_w


def backward_lowrank(x, g_y, w, k: int, bases):
    """Algorithm 1, step by step.

    x_hat <- p(x); g_y_hat <- p(g_y); g_w_hat <- g_y_hat^T x_hat (sum over
    batch, blocks and bases); g_x_hat <- g_y_hat w; g_x~ <- p^{-1}(g_x_hat);
    g_w~ <- g_w_hat.
    """
    w = np.asarray(w, dtype=np.float64)
    x_hat = project(x, k, bases)
    gy_hat = project(g_y, k, bases)
    Cin, Cout = x_hat.shape[-1], gy_hat.shape[-1]
    g_w_hat = gy_hat.reshape(-1, Cout).T @ x_hat.reshape(-1, Cin)
    g_x_hat = gy_hat @ w                                # (..., r, Cin)
    g_x = expand(g_x_hat, k, bases)
    return g_x, g_w_hat


# --------------------------------------------------------------------------
# Variants of Algorithm 1 that a ViT needs around its token grid.  The paper
# does not describe them; each docstring states the reading taken.
# --------------------------------------------------------------------------
def backward_lowrank_projected(x_hat, g_y, w, k: int, bases):
    """Algorithm 1 from its second step on, with x_hat = p(x) (Eq. 3) handed in
    instead of x: the projection of x can be taken at forward time and only its
    r/k^2 coefficients kept.

    x_hat (B, H/k, W/k, r, Cx) in the order of `bases`; g_y (B, H, W, Cy).
    g_y_hat <- p(g_y); g_w <- g_y_hat^T x_hat; g_x_hat <- g_y_hat w;
    g_x <- p^{-1}(g_x_hat).
    """
    _check_bases(k, bases)
    x_hat = np.asarray(x_hat, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    gy_hat = project(g_y, k, bases)
    if x_hat.shape[:4] != gy_hat.shape[:4]:
        raise ValueError("x_hat does not match the block grid of g_y")
    Cin, Cout = x_hat.shape[-1], gy_hat.shape[-1]
    g_w = gy_hat.reshape(-1, Cout).T @ x_hat.reshape(-1, Cin)
    g_x = expand(gy_hat @ w, k, bases)
    return g_x, g_w


def pad_grid(t, k: int) -> np.ndarray:
    """Reading for token grids whose sides are not multiples of the order k (the
    paper's 7 x 7 maps, L = 49, under an order-8 transform): the grid is
    extended with zero tokens at its high end (bottom rows, right columns) to
    the next multiple of k; blocks stay aligned at the origin."""
    t = np.asarray(t, dtype=np.float64)
    B, H, W, C = t.shape
    Hp, Wp = -(-H // k) * k, -(-W // k) * k
    out = np.zeros((B, Hp, Wp, C), dtype=np.float64)
    out[:, :H, :W, :] = t
    return out


def project_padded(t, k: int, bases) -> np.ndarray:
    """Eq. 6 on the zero-extended grid: (B,H,W,C) -> (B, ceil(H/k), ceil(W/k), r, C)."""
    return project(pad_grid(t, k), k, bases)


def backward_lowrank_padded(x, g_y, w, k: int, bases):
    """Algorithm 1 on the zero-extended grid; g_x is returned for the real tokens
    only (the gradient of a padding token has no consumer).  The zero tokens add
    nothing to g_w."""
    x = np.asarray(x, dtype=np.float64)
    B, H, W, _ = x.shape
    g_x, g_w = backward_lowrank(pad_grid(x, k), pad_grid(g_y, k), w, k, bases)
    return g_x[:, :H, :W, :], g_w


def backward_extra_tokens(x_extra, gy_extra, w):
    """Tokens that are not part of the grid (a class token): the paper's method
    has nothing to say about them, so they take vanilla BP (Eq. 2) exactly.
    x_extra (n, Cx), gy_extra (n, Cy) -> (g_x_extra (n, Cx), their term of g_w)."""
    x_extra = np.asarray(x_extra, dtype=np.float64)
    gy_extra = np.asarray(gy_extra, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    return gy_extra @ w, gy_extra.T @ x_extra


def bias_grad(g_y, gy_extra=None) -> np.ndarray:
    """Gradient of a bias added to y (Eq. 1 has none; every ViT linear has one):
    the sum of g_y over all tokens, exact.  For the grid tokens this equals
    k * sum over blocks of the (0,0) coefficient of g_y_hat."""
    g_y = np.asarray(g_y, dtype=np.float64)
    out = g_y.reshape(-1, g_y.shape[-1]).sum(axis=0)
    if gy_extra is not None:
        gy_extra = np.asarray(gy_extra, dtype=np.float64)
        out = out + gy_extra.reshape(-1, gy_extra.shape[-1]).sum(axis=0)
    return out


def accumulate(g_w_new, g_w_prev=None, beta: float = 0.0) -> np.ndarray:
    """g_w <- beta * g_w_prev + g_w_new (gradient accumulation over micro-batches)."""
    g_w_new = np.asarray(g_w_new, dtype=np.float64)
    if g_w_prev is None or beta == 0.0:
        return g_w_new
    return beta * np.asarray(g_w_prev, dtype=np.float64) + g_w_new


# --------------------------------------------------------------------------
# Cost model (Table 1)
# --------------------------------------------------------------------------
def flops(Cx: int, Cy: int, L: int, r: int) -> dict:
    """Table 1: FLOPs of vanilla BP and of the LBP-WHT components."""
    return {
        "vanilla": 4.0 * Cx * Cy * L,
        "projection": float((Cx + Cy) * L * r),
        "lowrank_mm": 4.0 * Cx * Cy * r,
        "reverse_projection": float(Cx * L * r),
    }


def rel_fro(a, b) -> float:
    """||a - b||_F / ||b||_F with b the reference (float64)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b.ravel())
    num = np.linalg.norm((a - b).ravel())
    return float(num / den) if den > 0 else float(num)


def block_rel_fro(a, b, k: int) -> float:
    """Largest relative Frobenius error over the k x k token blocks of a
    (B,H,W,C) tensor (H, W multiples of k): a wrong patch cannot hide in the
    norm of the whole tensor.  Blocks whose reference is all zero count with
    their absolute error."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = to_blocks(a - b, k)
    num = np.sqrt(np.sum(d * d, axis=(3, 4)))
    rb = to_blocks(b, k)
    den = np.sqrt(np.sum(rb * rb, axis=(3, 4)))
    ratio = np.where(den > 0, num / np.where(den > 0, den, 1.0), num)
    return float(ratio.max())


def tile_rel_fro(a, b, tile: int = 128) -> float:
    """Largest relative Frobenius error over tile x tile pieces of a matrix
    (ragged edge pieces included)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    worst = 0.0
    for i in range(0, b.shape[0], tile):
        for j in range(0, b.shape[1], tile):
            worst = max(worst, rel_fro(a[i:i + tile, j:j + tile], b[i:i + tile, j:j + tile]))
    return worst
