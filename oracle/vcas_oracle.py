"""CPU oracle for the variance-controlled sampled backward of one linear layer (VCAS).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the CUDA
library is checked against.  It shares no code with the CUDA path, is never imported
by the product package, and must only be used from tests, the smoke check and the
CPU-baseline leg of the benchmark.

Everything is numpy in float64 on inputs read at their stored precision.  The one
exception is deliberate: keep probabilities are rounded to float32 before they decide
a mask bit or a rescale factor, because the CUDA library stores them as float32 and a
Bernoulli decision has to be taken in one precision on both sides.

Notation follows the paper: N data, T tokens per datum, R = N*T rows, a layer
Z = X theta^T with theta = W of shape [d_out, d_in], G = dY of shape [R, d_out],
rho / nu the keep ratios of SampleA / SampleW.

Parity status: there is no worked numeric example in the paper, so nothing here is
pinned against the authors' numbers.  Every function is pinned against mathematics
instead (dense backprop at ratio 1, brute-force enumeration of all masks, closed-form
variances, published Philox known-answer vectors); the tests that do so are
tests/test_oracle_*.py.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
# SC'11).  Written from the published round function: two 32x32->64 multiplies, the high
# halves xor the neighbouring counter words and the key, the key is bumped by Weyl
# constants every round.
# --------------------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)
_PHILOX_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)
_SHIFT32 = np.uint64(32)


def philox4x32_10(counter, key):
    """Ten Philox rounds on arrays of 128-bit counters.

    counter: four uint32-valued arrays (broadcastable), key: two uint32-valued arrays.
    Returns the four output words as uint32 arrays.
    """
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & _MASK32 for c in counter)
    k0, k1 = (np.asarray(k, dtype=np.uint64) & _MASK32 for k in key)
    for _ in range(10):
        prod0 = _PHILOX_M0 * c0          # < 2^64, exact in uint64
        prod1 = _PHILOX_M1 * c2
        hi0, lo0 = prod0 >> _SHIFT32, prod0 & _MASK32
        hi1, lo1 = prod1 >> _SHIFT32, prod1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK32, lo1, (hi0 ^ c3 ^ k1) & _MASK32, lo0
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return tuple(np.asarray(c, dtype=np.uint32) for c in (c0, c1, c2, c3))


def uniform24(seed: int, stream: int, idx):
    """The 24-bit uniform integer drawn for element `idx` of sampler `stream`.

    Contract of this repository (the paper only says "Bernoulli with randomness eps",
    Sec. 4.1): key = (low, high) halves of the 64-bit seed, counter =
    (idx low, idx high, stream, 0), output word 0, top 24 bits.
    stream 0 = SampleA (idx = datum), stream 1 = SampleW (idx = global row).
    """
    idx = np.asarray(idx, dtype=np.uint64)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    k0 = np.uint64(seed & 0xFFFFFFFF)
    k1 = np.uint64(seed >> 32)
    zero = np.zeros_like(idx)
    out0 = philox4x32_10((idx & _MASK32, idx >> _SHIFT32, zero + np.uint64(stream), zero),
                         (zero + k0, zero + k1))[0]
    return (out0 >> np.uint32(8)).astype(np.uint32)


def bernoulli_keep(p32, seed: int, stream: int, idx=None):
    """keep_i = [u_i < floor(p_i * 2^24)] with u_i = uniform24(seed, stream, i).

    p32 must be float32 (the precision in which the decision is taken).  p = 1 always
    keeps (threshold 2^24 exceeds every u), p = 0 never keeps.
    """
    p32 = np.asarray(p32)
    assert p32.dtype == np.float32, "mask decisions are taken on float32 probabilities"
    if idx is None:
        idx = np.arange(p32.shape[0], dtype=np.uint64)
    # p * 2^24 is exact in float32 (power-of-two scale), so is its floor.
    thr = np.floor(p32.astype(np.float64) * 16777216.0).astype(np.uint32)
    return uniform24(seed, stream, idx) < thr


def probe_seed(seed: int, i: int, j: int, M: int) -> int:
    """Seed of Monte-Carlo repetition (i, j) of the probe (0-based), odd-constant stride."""
    return (int(seed) + (i * M + j + 1) * 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF


# --------------------------------------------------------------------------------------
# Scores and keep probabilities (Sec. 4.1, Sec. 4.2)
# --------------------------------------------------------------------------------------
def row_sqnorms(M):
    """||M_r||_2^2 for every row r (Sec. 4.2: token-wise 2-norms)."""
    M = np.asarray(M, dtype=np.float64)
    return np.sum(M * M, axis=1)


def datum_norms(a, N: int, T: int):
    """||G_n||_F for every datum n from the row square-norms a (Sec. 4.1)."""
    return np.sqrt(np.asarray(a, dtype=np.float64).reshape(N, T).sum(axis=1))


def capped_prop(v, budget: float):
    """Keep probabilities proportional to v, capped at 1, summing to the budget.

    Sec. 4.1 / 4.2 ask for p_i proportional to the score with sum p = budget; a plain
    proportional rule can exceed 1, so this is the minimiser of sum (1-p_i)/p_i v_i^2
    under sum p = budget, 0 <= p <= 1: p_i = min(1, c v_i) with c fixed by the budget
    (water-filling).  Zero scores get p = 0.  If the budget covers every non-zero
    score, all of those get p = 1.
    """
    v = np.asarray(v, dtype=np.float64)
    assert np.all(v >= 0.0)
    p = np.zeros_like(v)
    nz = int(np.count_nonzero(v))
    if nz == 0 or budget <= 0.0:
        return p
    if nz <= budget:
        p[v > 0.0] = 1.0
        return p
    order = np.argsort(-v, kind="stable")
    vs = v[order]
    # tail[k] = sum of the scores not among the k largest
    tail = np.cumsum(vs[::-1])[::-1]
    k = 0
    while True:
        c = (budget - k) / tail[k]
        if c * vs[k] <= 1.0:
            break
        k += 1
    p[order[:k]] = 1.0
    p[order[k:]] = c * vs[k:]
    return p


# --------------------------------------------------------------------------------------
# The samplers and the sampled backward (Eq. 2)
# --------------------------------------------------------------------------------------
def apply_data_mask(G, p, keep, T: int):
    """G_hat = G o (m x 1 x 1) with m_n = keep_n / p_n (Sec. 4.1); rows of dropped data are 0."""
    G = np.asarray(G, dtype=np.float64)
    keep = np.asarray(keep, dtype=bool)
    m = np.zeros(keep.shape[0], dtype=np.float64)
    m[keep] = 1.0 / np.asarray(p, dtype=np.float64)[keep]
    return G * np.repeat(m, T)[:, None]


def apply_row_mask(G_hat, q, keep):
    """G_tilde = G_hat o (m^T 1) with m_r = keep_r / q_r (Sec. 4.2)."""
    G_hat = np.asarray(G_hat, dtype=np.float64)
    keep = np.asarray(keep, dtype=bool)
    m = np.zeros(keep.shape[0], dtype=np.float64)
    m[keep] = 1.0 / np.asarray(q, dtype=np.float64)[keep]
    return G_hat * m[:, None]


def sample_a(dY, N: int, T: int, rho: float, seed: int, p_override=None):
    """SampleA (Sec. 4.1): data-dimension importance sampling of G = dY.

    p_n proportional to ||G_n||_F with sum p = N rho, mask from Philox stream 0.
    Returns dict(a, g, p32, keepA, G_hat).
    """
    dY = np.asarray(dY, dtype=np.float64)
    a = row_sqnorms(dY)
    g = datum_norms(a, N, T)
    if p_override is None:
        p32 = capped_prop(g, N * rho).astype(np.float32)
    else:
        p32 = np.asarray(p_override, dtype=np.float32)
    keepA = bernoulli_keep(p32, seed, 0)
    return dict(a=a, g=g, p32=p32, keepA=keepA, G_hat=apply_data_mask(dY, p32, keepA, T))


def sample_w(G_hat, X, keepA, N: int, T: int, nu: float, seed: int, q_override=None):
    """SampleW (Sec. 4.2): token-dimension leverage-score sampling of G_hat.

    Scores w_r = ||G_hat_r|| ||X_r|| (Eq. 3's minimiser), budget nu * T * #kept data
    (the keep ratio nu applies to the rows that survived SampleA; equal to the paper's
    N T rho nu in expectation).  Returns dict(w, q32, keepW, G_tilde).
    """
    G_hat = np.asarray(G_hat, dtype=np.float64)
    X = np.asarray(X, dtype=np.float64)
    w = np.sqrt(row_sqnorms(G_hat)) * np.sqrt(row_sqnorms(X))
    if q_override is None:
        q32 = capped_prop(w, nu * T * int(np.count_nonzero(keepA))).astype(np.float32)
    else:
        q32 = np.asarray(q_override, dtype=np.float32)
    keepW = bernoulli_keep(q32, seed, 1)
    return dict(w=w, q32=q32, keepW=keepW, G_tilde=apply_row_mask(G_hat, q32, keepW))


def linear_bwd(X, dY, W, N: int, T: int, rho: float, nu: float, seed: int,
               p_override=None, q_override=None):
    """Sampled backward of Z = X W^T (Eq. 2): dX = G_hat W, dW = G_tilde^T X."""
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    sa = sample_a(dY, N, T, rho, seed, p_override)
    sw = sample_w(sa["G_hat"], X, sa["keepA"], N, T, nu, seed, q_override)
    out = dict(sa)
    out.update(sw)
    out["b"] = row_sqnorms(X)
    out["dX"] = sa["G_hat"] @ W
    out["dW"] = sw["G_tilde"].T @ X
    out["idxA"] = np.flatnonzero(sa["keepA"]).astype(np.int32)
    out["idxW"] = np.flatnonzero(sw["keepW"]).astype(np.int32)
    return out


def dense_bwd(X, dY, W):
    """Exact backprop of the linear layer: dX = dY W, dW = dY^T X."""
    X = np.asarray(X, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    return dY @ W, dY.T @ X


def layernorm_bwd(X, gamma, dY, N: int, T: int, rho: float, seed: int, eps: float = 1e-5, p_override=None):
    """Backward of Y = LayerNorm(X) * gamma + beta over the last axis with SampleA in front of it
    (Eq. 2 for a layer without a weight-gradient sampler; App. E: the sampled, rescaled gradient G_hat is
    multiplied by the layer's exact Jacobian).  Returns dict(p32, keepA, dX, dgamma, dbeta, g).

    With x_hat = (x - mean) / sqrt(var + eps) per row and g_hat = G_hat * gamma:
      dX = (g_hat - mean(g_hat) - x_hat * mean(g_hat * x_hat)) / sqrt(var + eps)     (row-wise means),
      dgamma = sum_r G_hat_r * x_hat_r,   dbeta = sum_r G_hat_r.
    Rows of dropped data have G_hat = 0, hence dX = 0 and no contribution to dgamma, dbeta."""
    X = np.asarray(X, dtype=np.float64)
    gamma = np.asarray(gamma, dtype=np.float64)
    sa = sample_a(dY, N, T, rho, seed, p_override)
    G = sa["G_hat"]
    mean = X.mean(axis=1, keepdims=True)
    var = ((X - mean) ** 2).mean(axis=1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xh = (X - mean) * rstd
    gh = G * gamma
    dX = (gh - gh.mean(axis=1, keepdims=True) - xh * (gh * xh).mean(axis=1, keepdims=True)) * rstd
    return dict(p32=sa["p32"], keepA=sa["keepA"], g=sa["g"], dX=dX, dgamma=(G * xh).sum(axis=0), dbeta=G.sum(axis=0))


# --------------------------------------------------------------------------------------
# Closed-form variances (Sec. 4.1 and Eq. 3)
# --------------------------------------------------------------------------------------
def var_sample_a(g, p):
    """Var[G_hat] = sum_n (1-p_n)/p_n ||G_n||_F^2 over data with p_n > 0 (Sec. 4.1)."""
    g = np.asarray(g, dtype=np.float64)
    p = np.asarray(p, dtype=np.float64)
    ok = p > 0.0
    return float(np.sum((1.0 - p[ok]) / p[ok] * g[ok] ** 2))


def var_sample_w(G_hat, X, q):
    """Eq. 3: sum_r (1-q_r)/q_r ||G_hat_r||^2 ||X_r||^2 over rows with q_r > 0."""
    q = np.asarray(q, dtype=np.float64)
    ok = q > 0.0
    return float(np.sum((1.0 - q[ok]) / q[ok] * row_sqnorms(G_hat)[ok] * row_sqnorms(X)[ok]))


# --------------------------------------------------------------------------------------
# Ratio adaptation (Sec. 5, Alg. 1, App. D)
# --------------------------------------------------------------------------------------
def sparsity_p(g, s: float) -> float:
    """Eq. 4: the smallest fraction n/N of data whose largest norms hold a share s of the total.

    n ranges over 1..N, as the sum over i = 1..n in Eq. 4 does: at least one datum is always
    kept, so p(0) = 1/N, and an all-zero gradient gives 1/N as well (every n meets 0 >= 0).
    """
    g = np.sort(np.asarray(g, dtype=np.float64))[::-1]
    total = 0.0
    for x in g:                      # sequential sum in descending order: the cumulative
        total += x                   # sum of all N terms equals the total bit for bit
    target = s * total
    cum, n = g[0], 1
    while cum < target:
        cum += g[n]
        n += 1
    return n / g.shape[0]


def param_subset(d_out: int, k: int, seed: int):
    """A uniformly random subset of k of the layer's d_out output features (rows of theta), ascending.

    App. D estimates the variances on a small random sample of the parameters.  Contract of this
    repository: feature i gets the Philox word of counter (i, 0, 2, 0) under the key (seed low, seed high)
    (sampler id 2), and the k features with the smallest words are taken (ties by index)."""
    idx = np.arange(d_out, dtype=np.uint64)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    zero = np.zeros_like(idx)
    u = philox4x32_10((idx, zero, zero + np.uint64(2), zero),
                      (zero + np.uint64(seed & 0xFFFFFFFF), zero + np.uint64(seed >> 32)))[0]
    order = np.lexsort((np.arange(d_out), u))            # by word, then by index
    return np.sort(order[:k]).astype(np.int64)


def variance_probe(Xs, dYs, W, N: int, T: int, rho: float, nu: float, s: float,
                   alpha: float, seed: int, param_rows=None):
    """The Monte-Carlo probe of Alg. 1 for one linear layer's parameter gradient.

    param_rows (App. D: the variances are estimated on a sample of the parameters): if given, V_s and V_act
    are taken over these rows of the parameter gradient only and scaled by d_out / len(param_rows) - an
    unbiased estimate of the full sums when the rows are a uniformly random subset.  V_w is analytic (Eq. 3)
    and needs no gradient.

    Xs, dYs: M batches.  For every batch i the exact gradient G_s,i = dY_i^T X_i; for
    every repetition j a SampleA-only gradient G_act,ij = G_hat_ij^T X_i and the analytic
    SampleW variance V_w,ij (Eq. 3) at ratio nu.  Returns V_s, V_act, V_w as Alg. 1
    defines them, and the averaged sparsity candidates p(s - alpha), p(s + alpha)
    (App. D), with s +- alpha clipped to [0, 1].
    """
    M = len(Xs)
    assert M >= 2 and len(dYs) == M
    W = np.asarray(W, dtype=np.float64)
    rows = slice(None) if param_rows is None else np.asarray(param_rows)
    scale = 1.0 if param_rows is None else W.shape[0] / len(param_rows)
    G_s = []
    v_act, v_w, p_lo, p_hi = 0.0, 0.0, 0.0, 0.0
    for i in range(M):
        X = np.asarray(Xs[i], dtype=np.float64)
        dY = np.asarray(dYs[i], dtype=np.float64)
        G_s.append((dY.T @ X)[rows])
        g = datum_norms(row_sqnorms(dY), N, T)
        p_lo += sparsity_p(g, max(0.0, s - alpha))
        p_hi += sparsity_p(g, min(1.0, s + alpha))
        for j in range(M):
            sd = probe_seed(seed, i, j, M)
            sa = sample_a(dY, N, T, rho, sd)
            G_act = (sa["G_hat"].T @ X)[rows]
            v_act += float(np.sum((G_act - G_s[i]) ** 2))
            w = np.sqrt(row_sqnorms(sa["G_hat"])) * np.sqrt(row_sqnorms(X))
            q32 = capped_prop(w, nu * T * int(np.count_nonzero(sa["keepA"]))).astype(np.float32)
            v_w += var_sample_w(sa["G_hat"], X, q32)
    mean = sum(G_s) / M
    V_s = sum(float(np.sum((G - mean) ** 2)) for G in G_s) / (M - 1)
    return dict(V_s=scale * V_s, V_act=scale * v_act / (M * M), V_w=v_w / (M * M), p_lo=p_lo / M, p_hi=p_hi / M)


def update_ratios(s, rho, nu, V_s, V_act, V_w, p_lo, p_hi, *, tau_act, tau_w, alpha, beta,
                  rho_min=0.0, nu_min=0.0):
    """One adaptation step of Alg. 1 on L layers (index 0 = layer 1, the lowest).

    Eq. 5: s moves by +alpha when the total SampleA variance is at least tau_act times the
    total SGD variance (sign(0) = +1), else by -alpha; clipped to [0, 1].
    Eq. 4 + App. D: p_l is the candidate computed at the side s moved to; rho_l is the
    running maximum of p_j over j <= l.
    Eq. 7 (read as: too much variance raises the keep ratio): nu_l <- min(1, nu_l / beta)
    when V_w,l >= tau_w V_s,l, else nu_l * beta.
    """
    V_s, V_act, V_w = (np.asarray(x, dtype=np.float64) for x in (V_s, V_act, V_w))
    up = float(V_act.sum()) - tau_act * float(V_s.sum()) >= 0.0
    s_new = min(1.0, max(0.0, s + (alpha if up else -alpha)))
    cand = np.asarray(p_hi if up else p_lo, dtype=np.float64)
    rho_new = np.maximum(np.maximum.accumulate(cand), rho_min)
    nu = np.asarray(nu, dtype=np.float64)
    raise_nu = V_w - tau_w * V_s >= 0.0
    nu_new = np.where(raise_nu, np.minimum(1.0, nu / beta), nu * beta)
    nu_new = np.maximum(nu_new, nu_min)
    return s_new, rho_new, nu_new


# --------------------------------------------------------------------------------------
# Bookkeeping used in reports
# --------------------------------------------------------------------------------------
def training_flops_reduction(bp_keep_ratio: float) -> float:
    """Sec. 6.1: with FP : BP = 1 : 2, keeping a share r of BP saves 1 - (1 + 2 r)/3."""
    return 1.0 - (1.0 + 2.0 * bp_keep_ratio) / 3.0


def gelu_prime(h):
    """Derivative of the exact (erf) GELU: Phi(h) + h phi(h) (the saved Jacobian of App. E)."""
    from math import erf, sqrt, pi
    h = np.asarray(h, dtype=np.float64)
    Phi = 0.5 * (1.0 + np.vectorize(erf)(h / sqrt(2.0)))
    phi = np.exp(-0.5 * h * h) / sqrt(2.0 * pi)
    return Phi + h * phi


# --------------------------------------------------------------------------------------
# Entry-by-entry forms for inputs too large for the whole-matrix functions above
# --------------------------------------------------------------------------------------
def row_sqnorms_chunked(M, chunk: int = 2048):
    """row_sqnorms on slices of rows (same sums; avoids a float64 copy of a very large matrix)."""
    return np.concatenate([row_sqnorms(np.asarray(M[i:i + chunk], dtype=np.float64))
                           for i in range(0, M.shape[0], chunk)])


def dX_rows(dY, W, p32, keepA, T: int, rows):
    """Rows `rows` of dX = G_hat W (App. E): (1/p_n) dY_r W for rows of kept data, 0 otherwise."""
    W = np.asarray(W, dtype=np.float64)
    out = np.zeros((len(rows), W.shape[1]))
    for i, r in enumerate(rows):
        n = r // T
        if keepA[n]:
            out[i] = (np.asarray(dY[r], dtype=np.float64) / float(p32[n])) @ W
    return out


def dW_rows(dY, X, p32, q32, keepW, T: int, outs):
    """Rows `outs` of dW = G_tilde^T X (Sec. 4.2): sum over kept rows r of dY[r, o] / (p_n q_r) * X_r."""
    kept = np.flatnonzero(keepW)
    scale = 1.0 / (np.asarray(p32, dtype=np.float64)[kept // T] * np.asarray(q32, dtype=np.float64)[kept])
    Xk = np.asarray(X[kept], dtype=np.float64)
    out = np.zeros((len(outs), Xk.shape[1]))
    for i, oo in enumerate(outs):
        out[i] = (np.asarray(dY[kept, oo], dtype=np.float64) * scale) @ Xk
    return out


def scores_and_masks_large(X, dY, N: int, T: int, rho: float, nu: float, seed: int, p_override=None,
                           q_override=None, chunk: int = 2048):
    """Steps of sample_a / sample_w that precede the products, without forming G_hat: the row norm of
    G_hat_r is ||dY_r|| / p_n on rows of kept data and 0 elsewhere (Sec. 4.1), so the leverage scores of
    Sec. 4.2 follow from the row square-norms.  Returns dict(a, b, g, p32, keepA, w, q32, keepW)."""
    a = row_sqnorms_chunked(dY, chunk)
    b = row_sqnorms_chunked(X, chunk)
    g = datum_norms(a, N, T)
    p32 = capped_prop(g, N * rho).astype(np.float32) if p_override is None else np.asarray(p_override, np.float32)
    keepA = bernoulli_keep(p32, seed, 0)
    inv = np.zeros(N)
    inv[keepA] = 1.0 / p32[keepA].astype(np.float64)
    w = np.sqrt(a) * np.repeat(inv, T) * np.sqrt(b)
    if q_override is None:
        q32 = capped_prop(w, nu * T * int(np.count_nonzero(keepA))).astype(np.float32)
    else:
        q32 = np.asarray(q_override, dtype=np.float32)
    keepW = bernoulli_keep(q32, seed, 1)
    return dict(a=a, b=b, g=g, p32=p32, keepA=keepA, w=w, q32=q32, keepW=keepW)


def products_on_kept_rows(X, dY, W, p32, q32, keepA, keepW, T: int):
    """dX = G_hat W and dW = G_tilde^T X (Eq. 2) computed from the kept rows alone: every other row of
    G_hat and of G_tilde is zero by definition (Sec. 4.1, 4.2), so it contributes a zero row to dX and
    nothing to dW.  Returns (dX [R, d_in], dW [d_out, d_in])."""
    W = np.asarray(W, dtype=np.float64)
    p = np.asarray(p32, dtype=np.float64)
    q = np.asarray(q32, dtype=np.float64)
    rowsA = np.flatnonzero(np.repeat(np.asarray(keepA, dtype=bool), T))
    dX = np.zeros((dY.shape[0], W.shape[1]))
    G_hat = np.asarray(dY[rowsA], dtype=np.float64) * (1.0 / p[rowsA // T])[:, None]
    dX[rowsA] = G_hat @ W
    rowsW = np.flatnonzero(np.asarray(keepW, dtype=bool))
    G_tilde = np.asarray(dY[rowsW], dtype=np.float64) * (1.0 / p[rowsW // T])[:, None] * (1.0 / q[rowsW])[:, None]
    dW = G_tilde.T @ np.asarray(X[rowsW], dtype=np.float64)
    return dX, dW
