"""Pins of the oracle's dispatch report and of the two ablation switches: hand-worked cases and
invariants that tie the report to quantities computed another way."""
import json
import os

import numpy as np

import oracle as O
import workloads as W

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _pair_cost(R, groups, c):
    C = np.full((R, R), c["inter"], np.float32)
    for g in groups:
        for i in g:
            for j in g:
                C[i, j] = c["intra"]
    np.fill_diagonal(C, c["self"])
    return C


def test_report_hand_case():
    g = json.load(open(os.path.join(GOLD, "report_hand_case.json")))
    C = _pair_cost(g["R"], g["nodes"], g["cost"])
    B = O.default_preference(C)
    r = O.report(g["R"], g["E"], g["K"], g["e2r"], C, B, g["expert_load"], g["rank_load"], g["slot_expert"],
                 g["X"], g["lambda"])
    for key, want in g["expect"].items():
        got = r[key]
        if isinstance(want, list):
            assert list(got) == want, key
        elif isinstance(want, float):
            assert abs(got - want) <= 1e-15, (key, got, want)
        else:
            assert got == want, (key, got, want)


def test_report_marks_a_copy_hosted_by_the_home_rank():
    # one slot on rank 0 holding rank 0's own expert: neither intra nor inter, costs C[0][0] = 0
    R, E, K = 2, 2, 1
    C = np.array([[0, 2], [2, 0]], np.float32)
    r = O.report(R, E, K, [0, 1], C, O.default_preference(C), [10, 2], [10, 2], [0, -1], [[3, 0], [1, 0]], 3.0)
    assert r["slot_kind"].tolist() == [3, 0] and r["same_rank"] == 1 and r["clones"] == 1
    assert r["intra"] == 0 and r["inter"] == 0 and r["cost_ratio"] == 0.0 and r["cost_C"] == 0.0
    assert r["load_after"].tolist() == [10, 2]          # tokens left and re-entered the same rank
    assert r["rerouted"] == 4


def test_report_of_an_empty_plan_and_of_zero_load():
    R, E, K = 4, 4, 2
    C = _pair_cost(R, [[0, 1], [2, 3]], dict(self=0.0, intra=1.0, inter=3.0))
    B = O.default_preference(C)
    r = O.report(R, E, K, [0, 1, 2, 3], C, B, [4, 4, 4, 4], [4, 4, 4, 4], [-1] * 8, np.zeros((4, 8), np.int32))
    assert r["rho_before"] == 0.0 and r["rho_after"] == 0.0 and r["clones"] == 0 and r["rerouted"] == 0
    assert r["peak_reduction"] == 0.0 and r["hot_ranks"] == 0 and r["cold_ranks"] == 0
    z = O.report(R, E, K, [0, 1, 2, 3], C, B, [0] * 4, [0] * 4, [-1] * 8, np.zeros((4, 8), np.int32))
    assert all(z[k] == 0.0 for k in O.REPORT_REALS)     # zero denominators give 0, not NaN


def test_report_agrees_with_a_recount_of_the_rewritten_routing_table():
    """Part 3 (projected loads) must equal what one gets by counting, in the rewritten table, every
    entry at the rank that will execute it: the home rank of an expert index, the host of a slot."""
    cfg = W.get_config("cfg1").replace(L=3, seed=77)
    tk = W.routing_topk(cfg).numpy()
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode).numpy()
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group).numpy()
    B = O.default_preference(C)
    out = O.plan_layers(tk, cfg.R, cfg.E, cfg.K, e2r, C, cfg.eps, cfg.max_iters, cfg.tol)
    node = np.arange(cfg.R) // cfg.gpus_per_node
    for l in range(cfg.L):
        r = O.report(cfg.R, cfg.E, cfg.K, e2r, C, B, out["expert_load"][l], out["rank_load"][l],
                     out["slot_expert"][l], out["X"][l], 3.0)
        new = out["new_idx"][l].ravel()
        runs_on = np.where(new < cfg.E, e2r[np.minimum(new, cfg.E - 1)], (new - cfg.E) // cfg.K)
        recount = np.bincount(runs_on, minlength=cfg.R)
        assert (r["load_after"] == recount).all()
        assert r["rerouted"] == int((new >= cfg.E).sum()) == int(out["X"][l].sum())
        assert r["total_load"] == new.size and int(r["load_after"].sum()) == new.size
        assert (r["spill"] == O.spill(out["expert_load"][l], e2r, cfg.R, out["mean"][l])).all()
        assert r["hot_ranks"] == int((out["excess"][l] > 0).sum())
        assert r["cold_ranks"] == int((out["spare"][l] > 0).sum())
        # transfer kinds against the node layout of the generator
        se = out["slot_expert"][l].ravel()
        used = se >= 0
        home = e2r[np.maximum(se, 0)]; host = np.arange(cfg.S) // cfg.K
        assert r["intra"] == int((used & (home != host) & (node[home] == node[host])).sum())
        assert r["inter"] == int((used & (node[home] != node[host])).sum())
        assert r["cost_ratio"] == r["intra"] + 3.0 * r["inter"]
        assert abs(r["cost_C"] - float(C[home[used], host[used]].astype(np.float64).sum())) < 1e-9
        assert r["rho_after"] <= r["rho_before"] and 0.0 <= r["peak_reduction"] <= 1.0
        mean = new.size / cfg.R
        assert abs(r["rho_before"] - (out["rank_load"][l].max() - mean) / mean) < 1e-12


def test_ablation_switches_hand_case():
    g = json.load(open(os.path.join(GOLD, "ablation_hand_case.json")))
    R, E, K = g["R"], g["E"], g["K"]
    B = np.array(g["B"], np.float32)
    hint = np.array(g["plan_hint"], np.float32)
    zeroB, zeroT = np.zeros_like(B), np.zeros_like(hint)
    for name, (Bm, Tm) in dict(full=(B, hint), no_hint=(B, zeroT), no_topology=(zeroB, hint),
                               neither=(zeroB, zeroT)).items():
        m = O.match(R, E, K, g["e2r"], g["mean"], g["excess"], g["spill"], g["spare"], Bm, Tm)
        want = g["expect"][name]
        assert m["slot_expert"].tolist() == want["slot_expert"], name
        assert m["slot_tokens"].tolist() == want["slot_tokens"], name
        assert m["inner_rounds"] == want["inner_rounds"], name


def test_plan_layers_switches_feed_exact_zeros():
    """hint=False must equal a run whose plan is zero; topology=False one whose preference matrix is
    zero in Phase 2 only (Phase 3 keeps the real one)."""
    cfg = W.get_config("ladder16").replace(L=3, T=16 * 512)
    tk = W.routing_topk(cfg).numpy()
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode).numpy()
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group).numpy()
    B = O.default_preference(C)
    off = O.plan_layers(tk, cfg.R, cfg.E, cfg.K, e2r, C, cfg.eps, cfg.max_iters, cfg.tol, hint=False,
                        topology=False, do_assign=False)
    assert (off["plan"] == 0).all() and (off["n_iter"] == 0).all()
    for l in range(cfg.L):
        spl = O.spill(off["expert_load"][l], e2r, cfg.R, off["mean"][l])
        m = O.match(cfg.R, cfg.E, cfg.K, e2r, off["mean"][l], off["excess"][l], spl, off["spare"][l],
                    np.zeros_like(B), np.zeros((cfg.R, cfg.R), np.float32))
        a = O.auction(cfg.R, cfg.E, cfg.K, off["n"][l], m["slot_expert"], m["slot_tokens"], B)
        assert (off["slot_expert"][l].ravel() == m["slot_expert"]).all() and (off["X"][l] == a["X"]).all()


def test_one_hot_rank_workload_reaches_the_stated_imbalance():
    """The ladder workload sends the fraction rho_0/(R-1) of the tokens to one rank, which gives an
    initial imbalance of rho_0 in expectation (hot-rank load f N + (1-f) N / R against mean N / R)."""
    cfg = W.get_config("ladder32")
    tk = W.routing_topk(cfg).numpy()
    assert tk.shape == (cfg.L, cfg.T, cfg.k) and tk.min() >= 0 and tk.max() < cfg.E
    srt = np.sort(tk, axis=2)
    assert (srt[:, :, 1:] != srt[:, :, :-1]).all()                     # k distinct experts per token
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode).numpy()
    _, _, rl, _ = O.histogram(tk, cfg.R, cfg.E, e2r)
    rho = (rl.max(1) - rl.mean(1)) / rl.mean(1)
    want = np.array([0.1, 0.2, 0.3, 0.5, 0.7] * 3)
    assert np.abs(rho - want).max() < 0.06
