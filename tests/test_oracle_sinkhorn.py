"""Pins for the oracle's Phase-1 Sinkhorn solve (Appendix A.2).

Nothing here re-types the oracle's formula: the checks are closed forms, the marginal
constraints, symmetries of the problem, an independent LP solver and the paper's own
multiplicative statement of the iteration.
"""
import json
import math
import os

import numpy as np
import pytest
from scipy.optimize import linprog

import oracle as O
import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")
TINY = 1e-30        # eps0 small enough that the column cap is the identity


def _problem(rng, R, n_hot):
    """Integer supplies on n_hot ranks, integer demands on the others, equal totals."""
    perm = rng.permutation(R)
    hot, cold = perm[:n_hot], perm[n_hot:]
    s = np.zeros(R, np.float32); d = np.zeros(R, np.float32)
    s[hot] = rng.integers(1, 50, size=len(hot))
    tot = int(s.sum())
    cuts = np.sort(rng.integers(0, tot + 1, size=len(cold) - 1))
    d[cold] = np.diff(np.concatenate([[0], cuts, [tot]]))
    return s, d


def test_two_by_two_closed_form():
    g = json.load(open(os.path.join(GOLD, "two_by_two.json")))
    R = g["R"]
    C = np.zeros((R, R), np.float32)
    for key, val in g["C_entries"].items():
        i, j = map(int, key.split(","))
        C[i, j] = val                      # C is NOT symmetric: a transposed cost would change the answer
    r = O.sinkhorn(g["s"], g["d"], C, g["eps"], 500, eps0=TINY)
    T = r["plan"]
    for key in ("T02", "T03", "T12", "T13"):
        i, j = int(key[1]), int(key[2])
        assert T[i, j] == pytest.approx(g[key], rel=1e-12)
    assert T.sum() == pytest.approx(4.0, rel=1e-13)
    assert np.count_nonzero(T) == 4        # only hot rows x cold columns carry flow
    # the root really solves the quadratic
    th = math.exp(4.0); t = g["T02"]
    assert (1 - th) * t * t + (5 * th - 1) * t - 6 * th == pytest.approx(0.0, abs=1e-9)


def test_uniform_cost_is_rank_one_after_one_iteration():
    rng = np.random.default_rng(1)
    for R in (4, 9, 16):
        s, d = _problem(rng, R, R // 3 + 1)
        C = np.full((R, R), 2.5, np.float32)
        T = O.sinkhorn(s, d, C, 0.7, 1, eps0=TINY)["plan"]
        want = np.outer(s.astype(np.float64), d.astype(np.float64)) / d.sum()
        assert np.allclose(T, want, rtol=1e-13, atol=0)


def test_marginals_and_support():
    rng = np.random.default_rng(2)
    C = W.cost_matrix(16, 8, (0.0, 1.0, 10.0)).numpy()
    for trial in range(5):
        s, d = _problem(rng, 16, 5)
        r = O.sinkhorn(s, d, C, 0.5, 5000, tol=1e-13, eps0=TINY)
        T = r["plan"]
        assert (T >= 0).all()
        assert np.allclose(T.sum(0), d, rtol=1e-12)            # columns are exact after the v-update
        assert np.allclose(T.sum(1), s, rtol=1e-9, atol=1e-9)  # rows at convergence
        assert (T[s == 0, :] == 0).all() and (T[:, d == 0] == 0).all()
        assert r["row_err"] <= 1e-13 and not r["capped"]


def test_column_cap_never_exceeds_demand():
    rng = np.random.default_rng(3)
    C = W.cost_matrix(8, 4, (0.0, 1.0, 8.0)).numpy()
    s, d = _problem(rng, 8, 3)
    for iters in (1, 2, 7):
        T = O.sinkhorn(s, d, C, 0.4, iters)["plan"]             # default eps0 = 1e-8
        assert (T.sum(0) <= d + 1e-12).all()
        assert np.allclose(T.sum(0), d, rtol=1e-7)


def test_supply_scaling_when_supply_exceeds_demand():
    # sum s = 12 > sum d = 9: gamma = 0.75, the plan moves 9 tokens and rows are 0.75 * s
    C = W.cost_matrix(4, 2, (0.0, 1.0, 3.0)).numpy()
    s = np.array([8, 0, 4, 0], np.float32); d = np.array([0, 5, 0, 4], np.float32)
    r = O.sinkhorn(s, d, C, 1.0, 3000, tol=1e-14, eps0=TINY)
    T = r["plan"]
    assert np.allclose(T.sum(1), 0.75 * s, rtol=1e-10)
    assert np.allclose(T.sum(0), d, rtol=1e-12)
    # sum s < sum d: gamma = 1; columns are still normalised last, so they hold exactly
    r = O.sinkhorn(d[::-1].copy(), s[::-1].copy(), C, 1.0, 50, eps0=TINY)
    assert np.allclose(r["plan"].sum(0), s[::-1], rtol=1e-12)


def test_nothing_to_move():
    C = W.cost_matrix(4, 2, (0.0, 1.0, 3.0)).numpy()
    r = O.sinkhorn(np.zeros(4), np.zeros(4), C, 1.0, 10)
    assert (r["plan"] == 0).all() and r["n_iter"] == 0 and r["row_err"] == 0.0


def test_entropic_cost_approaches_the_lp_optimum():
    rng = np.random.default_rng(4)
    g = json.load(open(os.path.join(GOLD, "two_by_two.json")))
    for trial in range(6):
        R = int(rng.integers(4, 7))
        s, d = _problem(rng, R, int(rng.integers(1, R - 1)))
        C = rng.integers(1, 9, size=(R, R)).astype(np.float32)
        np.fill_diagonal(C, 0)
        hot = np.where(s > 0)[0]; cold = np.where(d > 0)[0]
        # independent LP: min <T, C> over the hot x cold block with equality marginals
        nh, nc = len(hot), len(cold)
        A = np.zeros((nh + nc, nh * nc)); b = np.concatenate([s[hot], d[cold]])
        for a in range(nh):
            A[a, a * nc:(a + 1) * nc] = 1
        for c in range(nc):
            A[nh + c, c::nc] = 1
        lp = linprog(C[np.ix_(hot, cold)].ravel().astype(np.float64), A_eq=A, b_eq=b, bounds=(0, None), method="highs")
        assert lp.status == 0
        prev = None
        for eps in (2.0, 0.5, 0.1):
            T = O.sinkhorn(s, d, C, eps, 40000, tol=1e-12, eps0=TINY)["plan"]
            cost = float((T * C).sum())
            gap = cost - lp.fun
            assert gap >= -1e-7
            assert gap <= eps * float(s.sum()) * math.log(nh * nc) + 1e-7
            if prev is not None:
                assert cost <= prev + 1e-7                      # decreasing in eps
            prev = cost
    # the golden 2x2 instance: LP optimum 6, entropic cost within 1.5e-5 at eps = 0.3
    C = np.zeros((4, 4), np.float32)
    for key, val in g["C_entries"].items():
        i, j = map(int, key.split(","))
        C[i, j] = val
    c03 = float((O.sinkhorn(g["s"], g["d"], C, 0.3, 20000, tol=1e-14, eps0=TINY)["plan"] * C).sum())
    assert 0 <= c03 - g["lp_optimum_cost"] < 2e-5


def test_kernel_ratio_drives_the_plan():
    # Two hot ranks on different nodes, two cold ranks each intra-node with one of them: on a
    # 2x2 positive kernel the cross ratio of the optimum diag(u) M diag(v) equals the cross ratio
    # of M itself, which is (M_intra / M_inter)^2 = exp(2 (lam - 1) / lam) at eps = lam.
    g = json.load(open(os.path.join(GOLD, "kernel_ratio.json")))
    lam = g["lambda"]
    assert g["ratio"] == pytest.approx(math.exp((lam - 1) / lam), rel=1e-15)
    C = W.cost_matrix(4, 2, (0.0, 1.0, lam)).numpy()
    s = np.array([3, 0, 0, 3], np.float32)                      # hot: rank 0 (node 0), rank 3 (node 1)
    d = np.array([0, 3, 3, 0], np.float32)                      # cold: rank 1 (node 0), rank 2 (node 1)
    T = O.sinkhorn(s, d, C, g["eps"], 4000, tol=1e-15, eps0=TINY)["plan"]
    cross = T[0, 1] * T[3, 2] / (T[0, 2] * T[3, 1])
    assert cross == pytest.approx(g["ratio"] ** 2, rel=1e-10)


def test_symmetries():
    rng = np.random.default_rng(5)
    R = 12
    C = W.cost_matrix(R, 4, (0.0, 1.0, 6.0)).numpy()
    s, d = _problem(rng, R, 4)
    base = O.sinkhorn(s, d, C, 0.6, 37, eps0=TINY)["plan"]      # NOT converged: symmetries hold per iterate
    # relabelling the ranks permutes the plan
    p = rng.permutation(R)
    Tp = O.sinkhorn(s[p], d[p], C[np.ix_(p, p)], 0.6, 37, eps0=TINY)["plan"]
    assert np.allclose(Tp, base[np.ix_(p, p)], rtol=1e-11, atol=1e-300)
    # scaling the masses scales the plan
    T3 = O.sinkhorn(4 * s, 4 * d, C, 0.6, 37, eps0=TINY)["plan"]
    assert np.allclose(T3, 4 * base, rtol=1e-12)
    # adding a constant to one column of C changes no iterate after its first v-update
    C2 = C.copy(); C2[:, 5] += 2.0
    conv = O.sinkhorn(s, d, C, 0.6, 20000, tol=1e-14, eps0=TINY)["plan"]
    conv2 = O.sinkhorn(s, d, C2, 0.6, 20000, tol=1e-14, eps0=TINY)["plan"]
    assert np.allclose(conv, conv2, rtol=1e-9, atol=1e-12)


def test_log_domain_equals_the_papers_multiplicative_iteration():
    rng = np.random.default_rng(6)
    C = W.cost_matrix(16, 8, (0.0, 1.0, 10.0)).numpy()
    for iters in (1, 2, 10, 200):
        s, d = _problem(rng, 16, 6)
        a = O.sinkhorn(s, d, C, 0.2, iters)["plan"]
        b = O.sinkhorn_gibbs(s, d, C, 0.2, iters)
        assert np.allclose(a, b, rtol=1e-10, atol=1e-290)


def test_first_update_uses_v_equal_one_on_every_rank():
    # After ONE iteration with a single cold column every row's flow is s_i * share, where the
    # shares follow u_i = s_i / sum_j M_ij over ALL ranks j (v starts at 1 everywhere), then the
    # column is normalised.  Checked through numpy, not through the oracle's own loop.
    C = W.cost_matrix(4, 2, (0.0, 1.0, 3.0)).numpy().astype(np.float64)
    s = np.array([5, 0, 2, 0], np.float32); d = np.array([0, 7, 0, 0], np.float32)
    T = O.sinkhorn(s, d, C.astype(np.float32), 1.0, 1, eps0=TINY)["plan"]
    M = np.exp(-C / 1.0)
    u = s / (M @ np.ones(4))
    w = u * M[:, 1]
    assert np.allclose(T[:, 1], 7 * w / w.sum(), rtol=1e-13)


def test_stopping_rule_and_history():
    rng = np.random.default_rng(7)
    C = W.cost_matrix(16, 8, (0.0, 1.0, 10.0)).numpy()
    s, d = _problem(rng, 16, 5)
    full = O.sinkhorn(s, d, C, 0.3, 400, history=True)
    h = full["err_hist"]
    assert len(h) == 400 and full["n_iter"] == 400
    tol = float(h[60]) * 1.0000001
    r = O.sinkhorn(s, d, C, 0.3, 400, tol=tol)
    first = int(np.argmax(h <= tol)) + 1
    assert r["n_iter"] == first and r["row_err"] == pytest.approx(h[first - 1], rel=1e-12)
    r5 = O.sinkhorn(s, d, C, 0.3, 400, tol=tol, check_every=7)
    assert r5["n_iter"] % 7 == 0 and r5["n_iter"] >= first and r5["n_iter"] < first + 7
    capped = O.sinkhorn(s, d, C, 0.3, 3, tol=1e-300)
    assert capped["capped"] and capped["n_iter"] == 3
    # the history is the row violation of the plan at that iteration (recomputed from the plan itself)
    T10 = O.sinkhorn(s, d, C, 0.3, 10, eps0=TINY)["plan"]
    assert np.abs(T10.sum(1) - s).sum() / s.sum() == pytest.approx(h[9], rel=1e-9)


def test_extreme_cost_over_eps_does_not_underflow():
    C = W.cost_matrix(16, 8, (0.0, 1.0, 12.0)).numpy()
    rng = np.random.default_rng(8)
    s, d = _problem(rng, 16, 4)
    r = O.sinkhorn(s, d, C, 0.005, 3000, tol=1e-12, eps0=TINY)   # C/eps up to 2400
    T = r["plan"]
    assert np.isfinite(T).all()
    assert np.allclose(T.sum(0), d, rtol=1e-12)
