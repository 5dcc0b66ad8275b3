"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that one plausible mistake in the oracle (dropped rescale, wrong
sign, transposed operand, wrong budget, off-by-one threshold) fails it.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import vcas_oracle as o


def rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------- Philox
def test_philox_known_answers(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = o.philox4x32_10([np.array([c]) for c in v[0:4]], [np.array([k]) for k in v[4:6]])
        assert [int(x[0]) for x in out] == v[6:10]


def test_uniform24_is_uniform_and_streams_differ():
    idx = np.arange(1 << 16)
    u0 = o.uniform24(7, 0, idx)
    u1 = o.uniform24(7, 1, idx)
    assert u0.max() < (1 << 24)
    assert np.mean(u0 == u1) < 1e-3
    # chi-square over 64 equal bins: 63 dof, mean 63, sd ~ 11.2
    counts = np.bincount(u0 >> 18, minlength=64)
    chi2 = np.sum((counts - len(idx) / 64) ** 2 / (len(idx) / 64))
    assert chi2 < 63 + 6 * 11.3
    # 64-bit seeds use both key words, 64-bit indices both counter words
    assert not np.array_equal(o.uniform24(1, 0, idx[:64]), o.uniform24(1 + (1 << 32), 0, idx[:64]))
    assert not np.array_equal(o.uniform24(1, 0, idx[:64]), o.uniform24(1, 0, idx[:64] + (1 << 32)))


def test_bernoulli_threshold_edges():
    p = np.array([0.0, 1.0, 0.5, 2.0 ** -24, 1.0 - 2.0 ** -24], dtype=np.float32)
    keeps = np.stack([o.bernoulli_keep(p, s, 0) for s in range(2000)])
    assert not keeps[:, 0].any()              # p = 0 never
    assert keeps[:, 1].all()                  # p = 1 always
    assert abs(keeps[:, 2].mean() - 0.5) < 4 * 0.5 / np.sqrt(2000)
    # strict '<' on the integer threshold: u < floor(p 2^24)
    u = o.uniform24(123, 1, np.arange(5))
    pp = ((u[2].astype(np.float64)) / 2 ** 24).astype(np.float32)   # threshold == u  -> dropped
    assert not o.bernoulli_keep(np.array([0, 0, pp, 0, 0], dtype=np.float32), 123, 1)[2]
    pp1 = ((u[2].astype(np.float64) + 1) / 2 ** 24).astype(np.float32)  # threshold == u+1 -> kept
    assert o.bernoulli_keep(np.array([0, 0, pp1, 0, 0], dtype=np.float32), 123, 1)[2]


def test_keep_frequency_matches_p_and_count_matches_sum_p():
    # E[#kept] = sum p = N rho (Sec. 4.1) and per-index keep frequency = p_i
    g = np.exp(1.5 * rng(0).standard_normal(48))
    p = o.capped_prop(g, 48 * 0.3).astype(np.float32)
    n_seeds = 4000
    keeps = np.stack([o.bernoulli_keep(p, s, 0) for s in range(n_seeds)])
    sd_count = np.sqrt(np.sum(p * (1 - p)) / n_seeds)
    assert abs(keeps.sum(1).mean() - 48 * 0.3) < 4 * sd_count + 1e-4
    sd_i = np.sqrt(p * (1 - p) / n_seeds) + 1e-6
    assert np.all(np.abs(keeps.mean(0) - p) < 5 * sd_i)


# ------------------------------------------------------------------------ capped_prop
@pytest.mark.parametrize("seed", range(6))
def test_capped_prop_invariants(seed):
    r = rng(seed)
    n = int(r.integers(3, 200))
    v = np.exp(2.0 * r.standard_normal(n))
    v[r.random(n) < 0.2] = 0.0
    budget = float(r.uniform(0.05, 0.95) * n)
    p = o.capped_prop(v, budget)
    nz = np.count_nonzero(v)
    assert np.all(p >= 0) and np.all(p <= 1)
    assert np.all(p[v == 0] == 0)
    assert np.isclose(p.sum(), min(budget, nz), rtol=1e-12)
    unsat = (p < 1) & (v > 0)
    if unsat.sum() > 1:
        ratio = p[unsat] / v[unsat]
        assert np.allclose(ratio, ratio[0], rtol=1e-12)
        # every saturated score is at least as large as every unsaturated one, and would exceed 1
        if (p == 1).any():
            assert v[p == 1].min() * ratio[0] >= 1.0 - 1e-12
    order = np.argsort(v)
    assert np.all(np.diff(p[order]) >= -1e-15)       # monotone in the score


def test_capped_prop_uniform_scores_give_rho():
    p = o.capped_prop(np.full(10, 3.7), 10 * 0.3)
    assert np.allclose(p, 0.3)


def test_capped_prop_budget_covers_all_nonzero():
    v = np.array([0.0, 2.0, 0.0, 1e-9, 5.0])
    assert np.array_equal(o.capped_prop(v, 3.0), np.array([0, 1, 0, 1, 1.0]))
    assert np.array_equal(o.capped_prop(v, 4.5), np.array([0, 1, 0, 1, 1.0]))
    assert np.array_equal(o.capped_prop(np.zeros(4), 2.0), np.zeros(4))


def test_capped_prop_minimises_variance_brute_force():
    # Sec. 4.1: p minimises sum (1-p_i)/p_i g_i^2 under sum p = budget, p <= 1.
    r = rng(5)
    for n, budget in [(4, 2.0), (5, 1.5), (6, 4.2)]:
        v = np.exp(1.5 * r.standard_normal(n))
        p = o.capped_prop(v, budget)
        best = np.sum((1 - p) / p * v ** 2)
        for _ in range(4000):
            x = r.dirichlet(np.ones(n)) * budget
            if np.any(x > 1) or np.any(x <= 0):
                continue
            assert np.sum((1 - x) / x * v ** 2) >= best - 1e-9 * abs(best)
        # and against a uniform keep probability
        u = np.full(n, budget / n)
        assert np.sum((1 - u) / u * v ** 2) >= best


def test_optimal_probabilities_are_proportional_to_norms():
    # p_n ~ ||G_n||_F (Sec. 4.1) and q_r ~ ||G_hat_r|| ||X_r|| (Sec. 4.2) on unsaturated entries
    r = rng(11)
    N, T, di, do = 6, 5, 7, 9
    dY = r.standard_normal((N * T, do)) * np.repeat(np.exp(r.standard_normal(N)), T)[:, None]
    X = r.standard_normal((N * T, di))
    W = r.standard_normal((do, di))
    out = o.linear_bwd(X, dY, W, N, T, 0.5, 0.5, seed=3)
    gn = np.sqrt((dY.reshape(N, T * do) ** 2).sum(1))
    assert np.allclose(out["g"], gn)
    un = out["p32"] < 1
    assert np.allclose((out["p32"] / gn)[un], (out["p32"] / gn)[un][0], rtol=1e-6)
    lev = np.linalg.norm(out["G_hat"], axis=1) * np.linalg.norm(X, axis=1)
    un = (out["q32"] < 1) & (out["q32"] > 0)
    assert un.sum() > 2
    assert np.allclose(out["q32"][un] / lev[un], out["q32"][un][0] / lev[un][0], rtol=1e-5)
    # budget of SampleW: nu * T * number of kept data
    assert np.isclose(out["q32"].sum(), 0.5 * T * out["keepA"].sum(), rtol=1e-5)
    assert np.all(out["q32"][np.repeat(~out["keepA"], T)] == 0)


# --------------------------------------------------------------------- exact backprop
def test_ratio_one_is_dense_backprop():
    r = rng(1)
    N, T, di, do = 5, 7, 11, 13
    X, dY, W = r.standard_normal((N * T, di)), r.standard_normal((N * T, do)), r.standard_normal((do, di))
    out = o.linear_bwd(X, dY, W, N, T, 1.0, 1.0, seed=99)
    assert out["keepA"].all() and out["keepW"].all()
    assert np.all(out["p32"] == 1) and np.all(out["q32"] == 1)
    # textbook backprop of Z = X W^T written with einsum (independent of the oracle's matmuls)
    assert np.allclose(out["dX"], np.einsum("ro,oi->ri", dY, W), rtol=1e-13, atol=1e-13)
    assert np.allclose(out["dW"], np.einsum("ro,ri->oi", dY, X), rtol=1e-13, atol=1e-13)
    dXd, dWd = o.dense_bwd(X, dY, W)
    assert np.allclose(dXd, out["dX"]) and np.allclose(dWd, out["dW"])
    assert dXd.shape == (N * T, di) and dWd.shape == (do, di)


def test_dense_bwd_is_the_gradient_of_the_layer():
    # finite differences of L = sum(Z o C), Z = X W^T  =>  dL/dX = C W, dL/dW = C^T X
    r = rng(2)
    X, W, C = r.standard_normal((4, 3)), r.standard_normal((5, 3)), r.standard_normal((4, 5))
    dX, dW = o.dense_bwd(X, C, W)
    eps = 1e-6
    for (i, j) in [(0, 0), (3, 2), (1, 1)]:
        Xp = X.copy(); Xp[i, j] += eps
        assert np.isclose((np.sum(Xp @ W.T * C) - np.sum(X @ W.T * C)) / eps, dX[i, j], rtol=1e-5)
    for (i, j) in [(0, 0), (4, 2), (2, 1)]:
        Wp = W.copy(); Wp[i, j] += eps
        assert np.isclose((np.sum(X @ Wp.T * C) - np.sum(X @ W.T * C)) / eps, dW[i, j], rtol=1e-5)


# ------------------------------------------------- brute force over all masks (exact)
def _tiny(seed, N, T, di, do):
    r = rng(seed)
    dY = r.standard_normal((N * T, do)) * np.repeat(np.exp(r.standard_normal(N)), T)[:, None]
    return r.standard_normal((N * T, di)), dY, r.standard_normal((do, di))


def test_sample_a_unbiased_and_variance_closed_form_brute_force():
    N, T, di, do = 4, 3, 5, 6
    X, dY, W = _tiny(3, N, T, di, do)
    g = o.datum_norms(o.row_sqnorms(dY), N, T)
    p = o.capped_prop(g, N * 0.5)
    dXd, dWd = o.dense_bwd(X, dY, W)
    mean_G = 0; mean_dX = 0; var_G = 0; var_dX = 0; var_dW = 0; mean_dW = 0
    for bits in itertools.product([0, 1], repeat=N):
        keep = np.array(bits, dtype=bool)
        pr = np.prod(np.where(keep, p, 1 - p))
        Gh = o.apply_data_mask(dY, p, keep, T)
        mean_G = mean_G + pr * Gh
        mean_dX = mean_dX + pr * (Gh @ W)
        mean_dW = mean_dW + pr * (Gh.T @ X)
        var_G += pr * np.sum((Gh - dY) ** 2)
        var_dX += pr * np.sum((Gh @ W - dXd) ** 2)
        var_dW += pr * np.sum((Gh.T @ X - dWd) ** 2)
    assert np.allclose(mean_G, dY, atol=1e-12)           # E[G_hat] = G
    assert np.allclose(mean_dX, dXd, atol=1e-12)         # App. E: linear layer keeps unbiasedness
    assert np.allclose(mean_dW, dWd, atol=1e-12)
    assert np.isclose(var_G, o.var_sample_a(g, p), rtol=1e-12)       # Sec. 4.1 closed form
    # by linearity the same form holds with G_n W and G_n^T X_n in place of G_n
    gW = np.sqrt(((dY @ W).reshape(N, -1) ** 2).sum(1))
    assert np.isclose(var_dX, o.var_sample_a(gW, p), rtol=1e-12)
    gX = np.array([np.linalg.norm(dY[n * T:(n + 1) * T].T @ X[n * T:(n + 1) * T]) for n in range(N)])
    assert np.isclose(var_dW, o.var_sample_a(gX, p), rtol=1e-12)


def test_sample_w_unbiased_and_eq3_brute_force():
    N, T, di, do = 3, 3, 4, 5          # R = 9 rows -> 512 masks
    X, dY, W = _tiny(4, N, T, di, do)
    p = np.array([0.5, 1.0, 0.25])
    keepA = np.array([True, True, False])
    Gh = o.apply_data_mask(dY, p, keepA, T)
    w = np.linalg.norm(Gh, axis=1) * np.linalg.norm(X, axis=1)
    q = o.capped_prop(w, 0.5 * T * keepA.sum())
    exact = Gh.T @ X
    mean = 0; var = 0
    rows = np.flatnonzero(q > 0)
    for bits in itertools.product([0, 1], repeat=len(rows)):
        keep = np.zeros(N * T, dtype=bool); keep[rows] = np.array(bits, dtype=bool)
        pr = np.prod(np.where(keep[rows], q[rows], 1 - q[rows]))
        dW = o.apply_row_mask(Gh, q, keep).T @ X
        mean = mean + pr * dW
        var += pr * np.sum((dW - exact) ** 2)
    assert np.allclose(mean, exact, atol=1e-12)                       # E[G_tilde] = G_hat
    assert np.isclose(var, o.var_sample_w(Gh, X, q), rtol=1e-12)      # Eq. 3
    # leverage-score q beats a uniform q of the same budget
    qu = np.where(q > 0, q.sum() / (q > 0).sum(), 0)
    assert o.var_sample_w(Gh, X, qu) >= o.var_sample_w(Gh, X, q)


def test_total_variance_decomposition_brute_force():
    # law of total variance (Sec. 5): Var = Var_eps[E_xi] + E_eps[Var_xi]
    N, T, di, do = 2, 2, 3, 3          # 4 data masks x up to 16 row masks
    X, dY, W = _tiny(6, N, T, di, do)
    g = o.datum_norms(o.row_sqnorms(dY), N, T)
    p = o.capped_prop(g, N * 0.6)
    exact = dY.T @ X
    total = 0; e_var_w = 0; var_a = 0
    for bits in itertools.product([0, 1], repeat=N):
        keepA = np.array(bits, dtype=bool)
        prA = np.prod(np.where(keepA, p, 1 - p))
        Gh = o.apply_data_mask(dY, p, keepA, T)
        var_a += prA * np.sum((Gh.T @ X - exact) ** 2)
        w = np.linalg.norm(Gh, axis=1) * np.linalg.norm(X, axis=1)
        q = o.capped_prop(w, 0.5 * T * keepA.sum())
        e_var_w += prA * o.var_sample_w(Gh, X, q)
        rows = np.flatnonzero(q > 0)
        for wb in itertools.product([0, 1], repeat=len(rows)):
            keepW = np.zeros(N * T, dtype=bool); keepW[rows] = np.array(wb, dtype=bool)
            prW = np.prod(np.where(keepW[rows], q[rows], 1 - q[rows]))
            total += prA * prW * np.sum((o.apply_row_mask(Gh, q, keepW).T @ X - exact) ** 2)
    assert np.isclose(total, var_a + e_var_w, rtol=1e-12)


# ------------------------------------------------------ Monte-Carlo through the seeds
def test_seeded_estimator_converges_at_inverse_sqrt_n():
    # mean over n seeds of the sampled gradients -> exact gradients, squared error ~ V / n
    N, T, di, do = 8, 4, 6, 5
    X, dY, W = _tiny(7, N, T, di, do)
    dXd, dWd = o.dense_bwd(X, dY, W)
    n_max = 10000
    acc_dX = np.zeros_like(dXd); acc_dW = np.zeros_like(dWd)
    errs = {}
    v_dW = 0.0
    for s in range(n_max):
        out = o.linear_bwd(X, dY, W, N, T, 0.5, 0.5, seed=s)
        acc_dX += out["dX"]; acc_dW += out["dW"]
        v_dW += np.sum((out["dW"] - dWd) ** 2)
        if s + 1 in (100, 1000, 10000):
            errs[s + 1] = (np.sum((acc_dX / (s + 1) - dXd) ** 2), np.sum((acc_dW / (s + 1) - dWd) ** 2))
    p = out["p32"].astype(np.float64)
    gW = np.sqrt(((dY @ W).reshape(N, -1) ** 2).sum(1))
    V_dX = o.var_sample_a(gW, p)
    V_dW = v_dW / n_max
    for n, (e_dX, e_dW) in errs.items():
        # E[err] = V / n; the squared error of a mean of many terms is within a small factor
        assert 0.2 * V_dX / n < e_dX < 4 * V_dX / n, (n, e_dX, V_dX / n)
        assert 0.2 * V_dW / n < e_dW < 4 * V_dW / n, (n, e_dW, V_dW / n)
    # slope -1 on a log-log plot between n = 100 and n = 10000
    slope = np.log(errs[10000][1] / errs[100][1]) / np.log(100.0)
    assert -1.5 < slope < -0.5


def test_seeded_kept_counts_match_budgets():
    N, T, di, do = 16, 8, 4, 4
    X, dY, W = _tiny(8, N, T, di, do)
    nA = []; nW = []; sumq = []
    for s in range(1500):
        out = o.linear_bwd(X, dY, W, N, T, 0.5, 0.25, seed=s)
        nA.append(out["keepA"].sum()); nW.append(out["keepW"].sum()); sumq.append(out["q32"].sum())
    assert abs(np.mean(nA) - N * 0.5) < 0.15                    # N rho
    assert abs(np.mean(nW) - np.mean(sumq)) < 0.3               # E[#rows] = E[sum q]
    assert abs(np.mean(nW) - N * T * 0.5 * 0.25) < 0.5          # N T rho nu in expectation


# ------------------------------------------------------------------------------ probe
def test_probe_definitions():
    r = rng(9)
    N, T, di, do, M = 6, 4, 5, 4, 3
    W = r.standard_normal((do, di))
    Xs = [r.standard_normal((N * T, di)) for _ in range(M)]
    dYs = [r.standard_normal((N * T, do)) * np.repeat(np.exp(r.standard_normal(N)), T)[:, None] for _ in range(M)]
    out = o.variance_probe(Xs, dYs, W, N, T, 0.5, 0.5, s=0.8, alpha=0.05, seed=5)
    # V_s: textbook unbiased sample variance of the M exact gradients, summed over entries
    Gs = np.stack([dY.T @ X for X, dY in zip(Xs, dYs)])
    assert np.isclose(out["V_s"], np.var(Gs, axis=0, ddof=1).sum(), rtol=1e-12)
    # V_act, V_w recomputed term by term from the samplers
    v_act = 0; v_w = 0
    for i in range(M):
        for j in range(M):
            sa = o.sample_a(dYs[i], N, T, 0.5, o.probe_seed(5, i, j, M))
            v_act += np.sum((sa["G_hat"].T @ Xs[i] - Gs[i]) ** 2) / M ** 2
            lev = np.linalg.norm(sa["G_hat"], axis=1) * np.linalg.norm(Xs[i], axis=1)
            q = o.capped_prop(lev, 0.5 * T * sa["keepA"].sum()).astype(np.float32).astype(np.float64)
            ok = q > 0
            v_w += np.sum((1 - q[ok]) / q[ok] * lev[ok] ** 2) / M ** 2
    assert np.isclose(out["V_act"], v_act, rtol=1e-12)
    assert np.isclose(out["V_w"], v_w, rtol=1e-12)
    seeds = {o.probe_seed(5, i, j, M) for i in range(M) for j in range(M)}
    assert len(seeds) == M * M and 5 not in seeds


def test_probe_sparsity_candidates_hand_case():
    """p_lo / p_hi of the probe (App. D): Eq. 4 at s - alpha and s + alpha, averaged over the M batches,
    with s -+ alpha clipped to [0, 1].  Norms are set by hand (T = 1, one non-zero entry per row), so the
    expected values below come from Eq. 4 by mental arithmetic, not from the oracle."""
    def batch(norms):
        dY = np.zeros((4, 3)); dY[:, 1] = norms
        return dY
    X = np.ones((4, 2)); W = np.ones((3, 2))
    # batch 0 norms 4 3 2 1 (total 10), batch 1 norms 8 1 .5 .5 (total 10); s = 0.7, alpha = 0.05
    #   s - alpha = 0.65: batch 0 needs 4 + 3 >= 6.5 -> 2/4;   batch 1: 8 >= 6.5 -> 1/4;   mean 0.375
    #   s + alpha = 0.75: batch 0 needs 4 + 3 + 2 >= 7.5 -> 3/4; batch 1: 8 >= 7.5 -> 1/4; mean 0.5
    dYs = [batch([3.0, 1.0, 4.0, 2.0]), batch([0.5, 8.0, 0.5, 1.0])]
    out = o.variance_probe([X, X], dYs, W, 4, 1, 0.5, 0.5, s=0.7, alpha=0.05, seed=0)
    assert out["p_lo"] == 0.375 and out["p_hi"] == 0.5
    # a swap of the two, a missing 1/M or a sum over the wrong side would give .5/.375, .75/1.0, ...
    # clip at the top: s + alpha = 1.03 -> 1: all non-zero data, 3/4 in both batches (unclipped, no n exists)
    dYs = [batch([3.0, 0.0, 4.0, 3.0]), batch([1.0, 8.0, 0.0, 1.0])]
    out = o.variance_probe([X, X], dYs, W, 4, 1, 0.5, 0.5, s=0.98, alpha=0.05, seed=0)
    assert out["p_hi"] == 0.75
    assert out["p_lo"] == 0.75                    # 0.93: 4 + 3 + 3 and 8 + 1 + 1 are needed
    # clip at the bottom: s - alpha < 0 -> 0: one datum (n >= 1); s + alpha = 0.07: the largest suffices
    out = o.variance_probe([X, X], dYs, W, 4, 1, 0.5, 0.5, s=0.02, alpha=0.05, seed=0)
    assert out["p_lo"] == 0.25 and out["p_hi"] == 0.25
    # three batches, unequal results: the mean is over M
    dYs = [batch([4.0, 3.0, 2.0, 1.0]), batch([8.0, 1.0, 0.5, 0.5]), batch([1.0, 1.0, 1.0, 1.0])]
    out = o.variance_probe([X, X, X], dYs, W, 4, 1, 0.5, 0.5, s=0.7, alpha=0.05, seed=0)
    assert np.isclose(out["p_lo"], (0.5 + 0.25 + 0.75) / 3) and np.isclose(out["p_hi"], (0.75 + 0.25 + 0.75) / 3)


def test_probe_v_act_approaches_closed_form():
    # E ||G_act - G_s||^2 = sum_n (1-p_n)/p_n ||G_n^T X_n||_F^2 (Sec. 4.1 form, by linearity)
    r = rng(10)
    N, T, di, do, M = 8, 3, 4, 4, 40
    W = r.standard_normal((do, di))
    X = r.standard_normal((N * T, di))
    dY = r.standard_normal((N * T, do)) * np.repeat(np.exp(r.standard_normal(N)), T)[:, None]
    out = o.variance_probe([X] * M, [dY] * M, W, N, T, 0.5, 0.5, s=1.0, alpha=0.01, seed=1)
    p = o.capped_prop(o.datum_norms(o.row_sqnorms(dY), N, T), N * 0.5).astype(np.float32).astype(np.float64)
    gX = np.array([np.linalg.norm(dY[n * T:(n + 1) * T].T @ X[n * T:(n + 1) * T]) for n in range(N)])
    assert np.isclose(out["V_act"], o.var_sample_a(gX, p), rtol=0.15)
    assert out["V_s"] < 1e-20                       # identical batches: no SGD variance


# ----------------------------------------------------------------------------- update
def test_sparsity_p_hand_cases():
    g = [1.0, 4.0, 2.0, 3.0]                        # sorted: 4 3 2 1, total 10
    assert o.sparsity_p(g, 0.7) == 0.5              # 4 + 3 = 7 >= 7
    assert o.sparsity_p(g, 0.71) == 0.75
    assert o.sparsity_p(g, 0.4) == 0.25
    assert o.sparsity_p(g, 1.0) == 1.0
    assert o.sparsity_p(g, 0.0) == 0.25             # n starts at 1: one datum is always kept
    assert o.sparsity_p(g, 0.39) == 0.25 and o.sparsity_p(g, 0.41) == 0.5
    assert o.sparsity_p([0.0, 5.0, 0.0, 0.0], 1.0) == 0.25     # only non-zero data are needed
    assert o.sparsity_p(np.zeros(3), 0.5) == 1 / 3             # 0 >= 0 holds from n = 1 on
    r = rng(12)
    g = np.exp(r.standard_normal(33))
    vals = [o.sparsity_p(g, s) for s in np.linspace(0, 1, 21)]
    assert np.all(np.diff(vals) >= 0)               # more norm preserved -> more data


def test_update_ratios_hand_cases(golden_dir):
    consts = dict(l.split() for l in open(os.path.join(golden_dir, "paper_constants.txt"))
                  if l.strip() and not l.startswith("#"))
    tau, alpha, beta = float(consts["tau"]), float(consts["alpha"]), float(consts["beta"])
    kw = dict(tau_act=tau, tau_w=tau, alpha=alpha, beta=beta)
    V_s = np.array([100.0, 100.0, 100.0])
    # SampleA variance 3*2 = 6 < 0.025*300 = 7.5 -> s goes down, candidates p_lo are used
    s, rho, nu = o.update_ratios(0.9, [1, 1, 1], [0.5, 0.5, 1.0], V_s, [2.0, 2.0, 2.0], [1.0, 2.5, 3.0],
                                 p_lo=[0.2, 0.1, 0.4], p_hi=[0.3, 0.2, 0.5], **kw)
    assert np.isclose(s, 0.89)
    assert np.allclose(rho, [0.2, 0.2, 0.4])        # running maximum from the lowest layer up
    # V_w: 1.0 < 2.5 -> lower nu; 2.5 >= 2.5 -> sign(0) = +1 raises nu; 3.0 raises, capped at 1
    assert np.allclose(nu, [0.5 * beta, 0.5 / beta, 1.0])
    # over budget: 9 >= 7.5 -> s goes up (variance-reducing direction), p_hi used
    s, rho, nu = o.update_ratios(0.9, [1, 1, 1], [0.5, 0.5, 1.0], V_s, [3.0, 3.0, 3.0], [1.0, 2.5, 3.0],
                                 p_lo=[0.2, 0.1, 0.4], p_hi=[0.3, 0.2, 0.5], **kw)
    assert np.isclose(s, 0.91) and np.allclose(rho, [0.3, 0.3, 0.5])
    # equality counts as +1 (Eq. 5's sign convention); s is clipped to [0, 1]
    s, _, _ = o.update_ratios(1.0, [1], [1], [40.0], [1.0], [0.0], [0.5], [0.6], **kw)
    assert s == 1.0
    s, _, _ = o.update_ratios(0.005, [1], [1], [40.0], [0.5], [0.0], [0.5], [0.6], **kw)
    assert s == 0.0
    # monotone schedule for arbitrary candidates
    r = rng(13)
    _, rho, _ = o.update_ratios(0.5, np.ones(24), np.ones(24), np.ones(24), np.ones(24), np.ones(24),
                                r.random(24), r.random(24), **kw)
    assert np.all(np.diff(rho) >= 0)


def test_flops_reduction_matches_paper(golden_dir):
    consts = dict(l.split() for l in open(os.path.join(golden_dir, "paper_constants.txt"))
                  if l.strip() and not l.startswith("#"))
    assert round(o.training_flops_reduction(1 / 3), 4) == float(consts["flops_reduction_at_one_third"])
    assert o.training_flops_reduction(1.0) == 0.0


def test_gelu_prime_is_the_derivative_of_gelu():
    import torch
    h = np.linspace(-4, 4, 41)
    t = torch.tensor(h, dtype=torch.float64, requires_grad=True)
    torch.nn.functional.gelu(t).sum().backward()          # library erf-GELU
    assert np.allclose(o.gelu_prime(h), t.grad.numpy(), rtol=1e-12, atol=1e-14)


def test_entrywise_forms_agree_with_whole_matrix_forms():
    # the per-row forms used on very large inputs are the same numbers as linear_bwd's matrices
    N, T, di, do = 6, 5, 7, 9
    X, dY, W = _tiny(21, N, T, di, do)
    out = o.linear_bwd(X, dY, W, N, T, 0.6, 0.5, seed=4)
    rows = [0, 7, 13, 29]
    assert np.allclose(o.dX_rows(dY, W, out["p32"], out["keepA"], T, rows), out["dX"][rows], rtol=1e-12, atol=1e-12)
    outs = [0, 3, 8]
    assert np.allclose(o.dW_rows(dY, X, out["p32"], out["q32"], out["keepW"], T, outs), out["dW"][outs],
                       rtol=1e-12, atol=1e-12)
    assert np.allclose(o.row_sqnorms_chunked(dY, chunk=4), o.row_sqnorms(dY), rtol=1e-15)


def test_kept_row_forms_agree_with_whole_matrix_forms():
    # the forms the full-size GPU tests use are the same numbers as linear_bwd's, with and without overrides
    N, T, di, do = 7, 6, 5, 8
    X, dY, W = _tiny(22, N, T, di, do)
    dY[2 * T:3 * T] = 0.0                                   # a datum dropped upstream
    for over in (False, True):
        ref = o.linear_bwd(X, dY, W, N, T, 0.6, 0.5, seed=9)
        kw = dict(p_override=ref["p32"] * np.float32(0.9), q_override=np.minimum(1, ref["q32"] * np.float32(1.1))) if over else {}
        ref = o.linear_bwd(X, dY, W, N, T, 0.6, 0.5, seed=9, **kw)
        sm = o.scores_and_masks_large(X, dY, N, T, 0.6, 0.5, 9, chunk=5, **kw)
        for k in ("a", "b", "g", "w"):
            assert np.allclose(sm[k], ref[k], rtol=1e-13, atol=0)
        for k in ("p32", "q32", "keepA", "keepW"):
            assert np.array_equal(sm[k], ref[k])
        dX, dW = o.products_on_kept_rows(X, dY, W, sm["p32"], sm["q32"], sm["keepA"], sm["keepW"], T)
        assert np.allclose(dX, ref["dX"], rtol=1e-12, atol=1e-13) and np.allclose(dW, ref["dW"], rtol=1e-12, atol=1e-13)
        assert 0 < sm["keepA"].sum() < N and 0 < sm["keepW"].sum() < sm["keepA"].sum() * T


def test_probe_on_a_parameter_subset_is_unbiased_for_the_full_sums():
    """App. D: variances estimated on a random sample of the parameters.  Averaged over ALL subsets of k of the
    d_out rows, the scaled subset estimates equal the full V_s and V_act exactly (each row is in the same
    share k/d_out of the subsets); V_w and the sparsity candidates do not depend on the subset."""
    r = rng(31)
    N, T, di, do, M, k = 5, 3, 4, 5, 2, 2
    W = r.standard_normal((do, di))
    Xs = [r.standard_normal((N * T, di)) for _ in range(M)]
    dYs = [r.standard_normal((N * T, do)) * np.repeat(np.exp(r.standard_normal(N)), T)[:, None] for _ in range(M)]
    full = o.variance_probe(Xs, dYs, W, N, T, 0.6, 0.5, s=0.8, alpha=0.05, seed=3)
    subs = list(itertools.combinations(range(do), k))
    outs = [o.variance_probe(Xs, dYs, W, N, T, 0.6, 0.5, s=0.8, alpha=0.05, seed=3, param_rows=list(c)) for c in subs]
    assert np.isclose(np.mean([x["V_s"] for x in outs]), full["V_s"], rtol=1e-12)
    assert np.isclose(np.mean([x["V_act"] for x in outs]), full["V_act"], rtol=1e-12)
    assert all(x["V_w"] == full["V_w"] and x["p_lo"] == full["p_lo"] and x["p_hi"] == full["p_hi"] for x in outs)
    assert len({round(x["V_s"], 9) for x in outs}) > 1                     # the subsets do differ
    # one subset, by hand: rows {1, 3} of the gradients, scaled by d_out / 2
    Gs = np.stack([dY.T @ X for X, dY in zip(Xs, dYs)])[:, [1, 3]]
    one = o.variance_probe(Xs, dYs, W, N, T, 0.6, 0.5, s=0.8, alpha=0.05, seed=3, param_rows=[1, 3])
    assert np.isclose(one["V_s"], do / 2 * np.var(Gs, axis=0, ddof=1).sum(), rtol=1e-12)


def test_param_subset_is_a_uniform_random_subset():
    k, d = 8, 40
    seen = np.zeros(d)
    for seed in range(3000):
        sub = o.param_subset(d, k, seed)
        assert len(sub) == k and len(set(sub)) == k and np.all(np.diff(sub) > 0) and 0 <= sub[0] and sub[-1] < d
        seen[sub] += 1
    expect = 3000 * k / d                               # every feature in a share k/d of the subsets
    chi2 = np.sum((seen - expect) ** 2 / (expect * (1 - k / d)))
    assert chi2 < (d - 1) + 6 * np.sqrt(2 * (d - 1))
    assert np.array_equal(o.param_subset(d, d, 5), np.arange(d))           # k = d: everything
    assert not np.array_equal(o.param_subset(d, k, 1), o.param_subset(d, k, 1 + (1 << 32)))   # both key words


def test_layernorm_bwd_is_autograd_at_ratio_one_and_unbiased():
    import torch
    r = rng(41)
    N, T, d = 4, 3, 6
    X = r.standard_normal((N * T, d)) * 2 + 0.5
    gamma, beta = r.standard_normal(d), r.standard_normal(d)
    dY = r.standard_normal((N * T, d)) * np.repeat(np.exp(r.standard_normal(N)), T)[:, None]
    # ratio 1: exact backward of the library LayerNorm (float64 autograd)
    xt = torch.tensor(X, requires_grad=True); gt = torch.tensor(gamma, requires_grad=True)
    bt = torch.tensor(beta, requires_grad=True)
    y = torch.nn.functional.layer_norm(xt, (d,), gt, bt, eps=1e-5)
    y.backward(torch.tensor(dY))
    out = o.layernorm_bwd(X, gamma, dY, N, T, 1.0, seed=0)
    assert out["keepA"].all()
    assert np.allclose(out["dX"], xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(out["dgamma"], gt.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(out["dbeta"], bt.grad.numpy(), rtol=1e-10, atol=1e-12)
    # sampled: all three are linear in G_hat, so the exact enumeration over the 2^N masks gives the exact backward
    g = o.datum_norms(o.row_sqnorms(dY), N, T)
    p = o.capped_prop(g, N * 0.5).astype(np.float32)
    mean = {k: 0 for k in ("dX", "dgamma", "dbeta")}
    for mask in itertools.product([0, 1], repeat=N):
        keep = np.array(mask, bool)
        pr = np.prod(np.where(keep, p.astype(np.float64), 1 - p.astype(np.float64)))
        G_hat = o.apply_data_mask(dY, p, keep, T)
        xt2 = torch.tensor(X, requires_grad=True); gt2 = torch.tensor(gamma, requires_grad=True)
        bt2 = torch.tensor(beta, requires_grad=True)
        torch.nn.functional.layer_norm(xt2, (d,), gt2, bt2, eps=1e-5).backward(torch.tensor(G_hat))
        for k, v in (("dX", xt2.grad), ("dgamma", gt2.grad), ("dbeta", bt2.grad)):
            mean[k] = mean[k] + pr * v.numpy()
    assert np.allclose(mean["dX"], xt.grad.numpy(), rtol=1e-9, atol=1e-12)
    assert np.allclose(mean["dgamma"], gt.grad.numpy(), rtol=1e-9, atol=1e-12)
    # one seeded call: dropped data give exactly zero rows, kept data carry 1/p
    out = o.layernorm_bwd(X, gamma, dY, N, T, 0.5, seed=3)
    keep = out["keepA"]
    assert 0 < keep.sum() < N
    assert not out["dX"][np.repeat(~keep, T)].any()
    xt3 = torch.tensor(X, requires_grad=True)
    torch.nn.functional.layer_norm(xt3, (d,), torch.tensor(gamma), torch.tensor(beta), eps=1e-5).backward(
        torch.tensor(o.apply_data_mask(dY, out["p32"], keep, T)))
    assert np.allclose(out["dX"], xt3.grad.numpy(), rtol=1e-10, atol=1e-12)
