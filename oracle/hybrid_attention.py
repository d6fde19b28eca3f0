"""Float64 CPU oracle for the hybrid attention forward pass (test infrastructure).

This module is TEST INFRASTRUCTURE.  It defines what "correct" means for the CUDA
library and is imported only by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  It shares no code with the CUDA path and never imports it.

What it follows (paper: "Attention Surgery", arXiv 2509.24899):

* Eq. 2 (softmax attention), the kernelised form of linear attention in the
  "Preliminaries: Linear Attention" section (the equation after Eq. 3, with the two
  sums that do not depend on the query index), and the hybrid attention equation of
  the "Hybrid Attention" section (label `eq:hybrid`), including the stabilising
  constant c_i and the token split T = T_S u T_L.
* The token rule T_S = { i | i mod R = 1 } (1-indexed), same section.
* The feature map phi of "Characterization of phi": an embedding network, its output
  split into P equal parts, part p raised to the power p, parts concatenated.

Readings taken where the paper is silent (each is restated next to the code):

* c_i is the maximum of the softmax-branch exponents only.  Two modes are provided:
  STAB_PAPER evaluates the equation exactly as printed (the linear terms are NOT
  multiplied by exp(-c_i)); STAB_EXACT multiplies the linear terms by exp(-c_i), which
  makes the result independent of c_i (weights exp(s_ij) next to phi_q.phi_k).
* The embedding network is `layers` linear maps, each followed by ReLU (also the last
  one, so that phi >= 0 as the paper requires), each with an optional bias added before
  the ReLU.  The activation choice itself is not fixed by the paper: parity unpinned for
  that choice (the pins fix everything else about phi: layer order, the inner ReLU, the
  bias placement and the powers are checked against hand-worked values).
* Rate 1 means every token is a softmax token; rate 0 means none is.
* With a spatial block (t, h, w) on the latent grid the 1-D rule is applied to the
  raster index inside each (clipped) block; with one block covering the whole grid
  this is exactly the paper's rule.

Everything is plain numpy in float64.  Query rows are independent, so they are
processed in row blocks to bound memory; no other blocking, fusion or reordering is
done.  Pure-Python loops are used in `hybrid_attention_bruteforce`, meant for tiny
inputs only.
"""
from __future__ import annotations

import math

import numpy as np

STAB_PAPER = 0
STAB_EXACT = 1


# --------------------------------------------------------------------------------------
# Token split ("Hybrid Attention": T_S = { i | i mod R = 1 }, 1-indexed)
# --------------------------------------------------------------------------------------
def softmax_token_mask(grid, block, rate):
    """Boolean mask [N] that is True for softmax tokens T_S.

    grid  = (T, Hg, Wg): latent grid; tokens are flattened row-major, w fastest.
    block = (bt, bh, bw): spatial block; blocks at the border are clipped to the grid.
    rate  = R: 1 -> all tokens, 0 -> none, else inside every block the tokens whose
            0-indexed raster position l (within the clipped block) has l mod R == 0,
            which is the paper's 1-indexed `i mod R = 1`.
    """
    T, Hg, Wg = (int(x) for x in grid)
    bt, bh, bw = (int(x) for x in block)
    R = int(rate)
    n = T * Hg * Wg
    if R == 0:
        return np.zeros(n, dtype=bool)
    if R == 1:
        return np.ones(n, dtype=bool)
    t, h, w = np.meshgrid(np.arange(T), np.arange(Hg), np.arange(Wg), indexing="ij")
    ot, oh, ow = (t // bt) * bt, (h // bh) * bh, (w // bw) * bw
    eh = np.minimum(bh, Hg - oh)
    ew = np.minimum(bw, Wg - ow)
    ell = ((t - ot) * eh + (h - oh)) * ew + (w - ow)
    return (ell % R == 0).reshape(n)


# --------------------------------------------------------------------------------------
# Feature map ("Characterization of phi")
# --------------------------------------------------------------------------------------
def phi_features(x, weights, degree=2):
    """phi(x) for x[..., d] with one head's embedding network.

    weights: one matrix, or a list with one entry per layer; an entry is a matrix W_l of shape
             [out_l, in_l] or a pair (W_l, b_l) with a bias vector b_l [out_l].  The network is
             a_0 = x, a_{l+1} = ReLU(W_l a_l + b_l)  (b_l = 0 when no bias is given).
    The last activation [..., F] is split into `degree` = P contiguous equal parts;
    part p (1-indexed) is raised elementwise to the power p; parts are concatenated.
    """
    a = np.asarray(x, dtype=np.float64)
    if isinstance(weights, np.ndarray):
        weights = [weights]
    for l, layer in enumerate(weights):
        W, b = layer if isinstance(layer, tuple) else (layer, None)
        a = a @ np.asarray(W, dtype=np.float64).T
        if b is not None:
            a = a + np.asarray(b, dtype=np.float64)
        a = np.maximum(a, 0.0)
    F = a.shape[-1]
    P = int(degree)
    if F % P != 0:
        raise ValueError("feature dim must be divisible by the polynomial degree")
    part = F // P
    out = np.empty_like(a)
    for p in range(P):
        out[..., p * part:(p + 1) * part] = a[..., p * part:(p + 1) * part] ** (p + 1)
    return out


# --------------------------------------------------------------------------------------
# Linear state: S = sum_{j in T_L} phi_k(k_j)^T v_j,  z = sum_{j in T_L} phi_k(k_j)
# --------------------------------------------------------------------------------------
def linear_state(k, v, wk, is_softmax, degree=2):
    """S [F, d] and z [F] for one (batch, head): sums over the linear tokens only."""
    lin = ~np.asarray(is_softmax, dtype=bool)
    fk = phi_features(k[lin], wk, degree)           # [N_L, F]
    S = fk.T @ v[lin]                                # [F, d]
    z = fk.sum(axis=0)                               # [F]
    return S, z


# --------------------------------------------------------------------------------------
# Hybrid attention, factorised evaluation of the hybrid equation
# --------------------------------------------------------------------------------------
def hybrid_attention_head(q, k, v, wq, wk, is_softmax, scale=None, stab_mode=STAB_PAPER,
                          degree=2, row_block=2048, rows=None):
    """One (batch, head).  q, k, v: [N, d] float64; wq, wk: [F, d] (or lists of layers).

    Returns (y [n_rows, d], aux [n_rows, 3]) with aux = (c_i, den_S, den_L):
      c_i   = max_{j in T_S} s_ij               (0 when T_S is empty)
      den_S = sum_{j in T_S} exp(s_ij - c_i)    (0 when T_S is empty)
      den_L = phi_q(q_i) . z                    (0 when T_L is empty), before lambda_i.
    y_i = (sum_{T_S} exp(s_ij - c_i) v_j + lambda_i phi_q(q_i) S)
          / (den_S + lambda_i den_L),
    lambda_i = 1 (STAB_PAPER) or exp(-c_i) (STAB_EXACT); lambda_i = 1 when T_S is empty.
    `rows` (optional) selects the query rows to evaluate.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    is_softmax = np.asarray(is_softmax, dtype=bool)
    N, d = q.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    if rows is None:
        rows = np.arange(N)
    rows = np.asarray(rows)
    n_s = int(is_softmax.sum())
    n_l = k.shape[0] - n_s
    k_s, v_s = k[is_softmax], v[is_softmax]
    if n_l > 0:
        S, z = linear_state(k, v, wk, is_softmax, degree)
    y = np.empty((len(rows), d))
    aux = np.zeros((len(rows), 3))
    for r0 in range(0, len(rows), row_block):
        idx = rows[r0:r0 + row_block]
        qb = q[idx]
        num = np.zeros((len(idx), d))
        den = np.zeros(len(idx))
        lam = np.ones(len(idx))
        if n_s > 0:
            s = (qb @ k_s.T) * scale                  # s_ij, j in T_S
            c = s.max(axis=1)                          # c_i
            e = np.exp(s - c[:, None])
            num += e @ v_s
            den_s = e.sum(axis=1)
            den += den_s
            aux[r0:r0 + len(idx), 0] = c
            aux[r0:r0 + len(idx), 1] = den_s
            if stab_mode == STAB_EXACT:
                lam = np.exp(-c)
            elif stab_mode != STAB_PAPER:
                raise ValueError("unknown stab_mode")
        if n_l > 0:
            fq = phi_features(qb, wq, degree)          # [rows, F]
            den_l = fq @ z
            num += lam[:, None] * (fq @ S)
            den += lam * den_l
            aux[r0:r0 + len(idx), 2] = den_l
        with np.errstate(invalid="ignore", divide="ignore"):
            y[r0:r0 + len(idx)] = num / den[:, None]
    return y, aux


def hybrid_attention(q, k, v, wq, wk, is_softmax, scale=None, stab_mode=STAB_PAPER,
                     degree=2, row_block=2048, rows=None):
    """All (batch, head) pairs.  q, k, v: [B, H, N, d]; wq, wk: [H, F, d].

    Returns (y [B, H, n_rows, d], aux [B, H, n_rows, 3]); see `hybrid_attention_head`.
    """
    q = np.asarray(q)
    B, H, N, d = q.shape
    n_rows = N if rows is None else len(rows)
    y = np.empty((B, H, n_rows, d))
    aux = np.empty((B, H, n_rows, 3))
    for b in range(B):
        for h in range(H):
            y[b, h], aux[b, h] = hybrid_attention_head(
                q[b, h], k[b, h], v[b, h], wq[h], wk[h], is_softmax, scale, stab_mode,
                degree, row_block, rows)
    return y, aux


# --------------------------------------------------------------------------------------
# Brute force: explicit N x N weights, scalar Python arithmetic, no S / z factorisation
# --------------------------------------------------------------------------------------
def hybrid_attention_bruteforce(q, k, v, wq, wk, is_softmax, scale=None,
                                stab_mode=STAB_PAPER, degree=2):
    """One head, tiny inputs.  Builds every weight w_ij with scalar loops:

      w_ij = exp(s_ij - c_i)                       if j in T_S
      w_ij = lambda_i * <phi_q(q_i), phi_k(k_j)>   if j in T_L
      y_i  = sum_j w_ij v_j / sum_j w_ij

    Returns (y [N, d], w [N, N]) with w already divided by its row sum.
    """
    q = [[float(x) for x in row] for row in np.asarray(q)]
    k = [[float(x) for x in row] for row in np.asarray(k)]
    v = [[float(x) for x in row] for row in np.asarray(v)]
    wq = [[float(x) for x in row] for row in np.asarray(wq)]
    wk = [[float(x) for x in row] for row in np.asarray(wk)]
    member = [bool(x) for x in np.asarray(is_softmax)]
    N, d = len(q), len(q[0])
    M = len(k)                       # number of keys
    F = len(wq)
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    part = F // degree

    def phi(x, W):
        out = []
        for f in range(F):
            a = 0.0
            for t in range(d):
                a += W[f][t] * x[t]
            a = a if a > 0.0 else 0.0
            out.append(a ** (f // part + 1))
        return out

    fq = [phi(x, wq) for x in q]
    fk = [phi(x, wk) for x in k]
    y = np.zeros((N, d))
    w = np.zeros((N, M))
    for i in range(N):
        s = {}
        for j in range(M):
            if member[j]:
                s[j] = scale * sum(q[i][t] * k[j][t] for t in range(d))
        c = max(s.values()) if s else 0.0
        lam = math.exp(-c) if (stab_mode == STAB_EXACT and s) else 1.0
        row = []
        for j in range(M):
            if member[j]:
                row.append(math.exp(s[j] - c))
            else:
                row.append(lam * sum(fq[i][f] * fk[j][f] for f in range(F)))
        tot = sum(row)
        for j in range(M):
            w[i, j] = row[j] / tot if tot != 0.0 else float("nan")
        for t in range(d):
            y[i, t] = sum(w[i, j] * v[j][t] for j in range(M))
    return y, w
