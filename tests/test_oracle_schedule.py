"""Pins for the oracle's Phase 2 (Algorithm 2), Phase 3 (Algorithm 3) and token reassignment.

Hand-derived special cases (each with its derivation in a comment), the hand trace stored in
golden/w1_hand_trace.json, and the constraints of Appendix A.3 / A.4 on seeded random inputs.
"""
import json
import os

import numpy as np
import pandas as pd
import pytest

import oracle as O
import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")
THIRD = np.float32(1.0) / np.float32(3.0)


def _two_node_B():
    # 4 ranks, 2 per node: 1 intra-node, 1/3 inter-node, 0 home
    C = W.cost_matrix(4, 2, (0.0, 1.0, 3.0)).numpy()
    B = O.default_preference(C)
    assert B[0, 1] == 1 and B[0, 2] == THIRD and B[0, 0] == 0
    return C, B


def test_default_preference_three_tiers():
    C = W.cost_matrix(64, 8, (0.0, 1.0, 6.0, 16.0), 4).numpy()
    B = O.default_preference(C)
    assert B[0, 0] == 0 and B[0, 1] == 1
    assert B[0, 8] == np.float32(1) / np.float32(6) and B[0, 32] == np.float32(1) / np.float32(16)


# ---------------------------------------------------------------------------- Phase 2


def _match_one(spill, spare, excess, B, plan, mean, K=1, R=4, E=4, e2r=None):
    e2r = np.arange(E, dtype=np.int32) * R // E if e2r is None else e2r
    return O.match(R, E, K, e2r, mean, np.array(excess, np.int32), np.array(spill, np.int32),
                   np.array(spare, np.int32), B, plan)


def test_match_topology_breaks_equal_gain():
    # expert 0 (home rank 0) spills 10; ranks 1 (same node) and 2 (other node) both have spare 10.
    # Both pick expert 0 with gain 10; alpha = 6*4/4 = 6; scores 10 + 6 vs 10 + 2: rank 1 wins the
    # arbitration, takes all 10, and nothing is left for rank 2.
    _, B = _two_node_B()
    m = _match_one([10, 0, 0, 0], [0, 10, 10, 0], [10, 0, 0, 0], B, np.zeros((4, 4), np.float32), mean=6)
    assert m["slot_expert"].tolist() == [-1, 0, -1, -1] and m["slot_tokens"].tolist() == [0, 10, 0, 0]
    assert m["inner_rounds"] == 1


def test_match_balance_gain_dominates_topology():
    # rank 1 (intra) has spare 2, rank 2 (inter) spare 10, expert 0 spills 10, alpha = 6:
    # rank 1 scores 2 + 6 = 8, rank 2 scores 10 + 2 = 12 -> rank 2 wins and takes 10.
    _, B = _two_node_B()
    m = _match_one([10, 0, 0, 0], [0, 2, 10, 0], [10, 0, 0, 0], B, np.zeros((4, 4), np.float32), mean=6)
    assert m["slot_expert"].tolist() == [-1, -1, 0, -1] and m["slot_tokens"].tolist() == [0, 0, 10, 0]


def test_match_ot_hint_breaks_the_remaining_tie():
    # ranks 2 and 3 are both inter-node for expert 0 with equal spare: gain and topology tie.
    # The hint T[0][3] = 7 > T[0][2] = 3 makes rank 3 win; with no hint the lowest rank wins.
    _, B = _two_node_B()
    plan = np.zeros((4, 4), np.float32); plan[0, 2] = 3; plan[0, 3] = 7
    m = _match_one([10, 0, 0, 0], [0, 0, 10, 10], [10, 0, 0, 0], B, plan, mean=6)
    assert m["slot_expert"].tolist() == [-1, -1, -1, 0]
    m = _match_one([10, 0, 0, 0], [0, 0, 10, 10], [10, 0, 0, 0], B, np.zeros((4, 4), np.float32), mean=6)
    assert m["slot_expert"].tolist() == [-1, -1, 0, -1]


def test_match_loser_reselects_in_the_same_outer_round():
    # R=4 (2 per node), E=8 (2 per rank).  Hot rank 0 spills e0 = 6 and e1 = 9; cold ranks 1, 2
    # have spare 9 and 8.  mean 8, alpha = 8*4/8 = 4.
    # round 1: rank 1: e1 -> min(9,9)+4 = 13, e0 -> 6+4 = 10: picks e1.  rank 2: e1 -> 8+4/3 = 9.33,
    #          e0 -> 6+1.33 = 7.33: picks e1.  Arbitration: rank 1 (13) beats rank 2 (9.33): g = 9.
    # round 2: rank 1 is matched; rank 2 now sees only e0 (e1 has spill 0): g = min(6, 8) = 6.
    _, B = _two_node_B()
    e2r = np.repeat(np.arange(4), 2).astype(np.int32)
    m = _match_one([6, 9, 0, 0, 0, 0, 0, 0], [0, 9, 8, 0], [15, 0, 0, 0], B, np.zeros((4, 4), np.float32),
                   mean=8, E=8, e2r=e2r)
    assert m["slot_expert"].tolist() == [-1, 1, 0, -1] and m["slot_tokens"].tolist() == [0, 9, 6, 0]
    assert m["inner_rounds"] == 2
    assert m["spill_left"].tolist() == [0] * 8 and m["spare_left"].tolist() == [0, 0, 2, 0]


def test_match_k_slots_and_no_duplicate_expert_on_a_rank():
    # one cold rank (1) with spare 20; hot rank 0 holds e0 (spill 5) and e1 (spill 7); K = 3.
    # kappa 0 takes e1 (gain 7 > 5), kappa 1 takes e0, kappa 2 finds nothing (both already placed there).
    _, B = _two_node_B()
    e2r = np.repeat(np.arange(4), 2).astype(np.int32)
    m = _match_one([5, 7, 0, 0, 0, 0, 0, 0], [0, 20, 0, 0], [12, 0, 0, 0], B, np.zeros((4, 4), np.float32),
                   mean=10, K=3, E=8, e2r=e2r)
    assert m["slot_expert"].reshape(4, 3)[1].tolist() == [1, 0, -1]
    assert m["slot_tokens"].reshape(4, 3)[1].tolist() == [7, 5, 0]


def test_w1_hand_trace_phase2_and_phase3():
    g = json.load(open(os.path.join(GOLD, "w1_hand_trace.json")))
    R, E = g["R"], g["E"]
    e2r = np.array(g["e2r"], np.int32)
    C = W.cost_matrix(R, g["gpus_per_node"], g["cost_tiers"]).numpy()
    B = O.default_preference(C)
    plan = np.zeros((R, R), np.float32)
    for key, val in g["converged_plan"].items():
        i, j = map(int, key.split(","))
        plan[i, j] = val
    n = np.tile(np.array(g["n_row_every_rank"], np.int32), (R, 1))
    alpha = np.float32(g["mean"] * R) / np.float32(E)
    assert alpha == g["alpha"]
    for K, key in ((1, "K1"), (2, "K2")):
        m = O.match(R, E, K, e2r, g["mean"], np.array(g["excess"], np.int32), np.array(g["spill"], np.int32),
                    np.array(g["spare"], np.int32), B, plan)
        assert m["slot_expert"].reshape(R, K).tolist() == (g[key]["slot_expert"] if K > 1 else [[x] for x in g[key]["slot_expert"]])
        assert m["slot_tokens"].reshape(R, K).tolist() == (g[key]["slot_tokens"] if K > 1 else [[x] for x in g[key]["slot_tokens"]])
    a = O.auction(R, E, 2, n, m["slot_expert"], m["slot_tokens"], B, price_step=0.1)
    want = np.zeros((R, R * 2), np.int32)
    for key, val in g["X_K2"].items():
        i, j = map(int, key.split(","))
        want[i, j] = val
    assert (a["X"] == want).all()
    assert a["rounds"] == g["auction_rounds_K2"] and a["residual"] == 0
    # imbalance after the plan
    load = np.array(g["rank_load"])
    for s in range(R * 2):
        e = m["slot_expert"][s]
        if e >= 0:
            load[e2r[e]] -= m["slot_tokens"][s]; load[s // 2] += m["slot_tokens"][s]
    assert (load.max() - g["mean"]) / g["mean"] == g["rho_after_K2"]


# ---------------------------------------------------------------------------- Phase 3


def test_auction_prefers_intra_node_then_lowest_rank():
    # one slot on rank 1 (node 0) for expert 0, wanting 5; holders: rank 0 has 4, ranks 2 and 3 have 3.
    # round 1: rank 0 (bonus 1) gives 4.  round 2: ranks 2, 3 tie at 1/3 -> rank 2 gives 1.
    _, B = _two_node_B()
    n = np.zeros((4, 4), np.int32); n[:, 0] = [4, 0, 3, 3]
    a = O.auction(4, 4, 1, n, [-1, 0, -1, -1], [0, 5, 0, 0], B)
    assert a["X"][:, 1].tolist() == [4, 0, 1, 0] and a["rounds"] == 2 and a["residual"] == 0


def test_auction_price_spreads_sources():
    # two slots on ranks 2 and 3 (node 1) for expert 0, each wanting 2; the same-node holders are
    # rank 2 and rank 3 themselves with 1 token each, node-0 ranks hold 10 each.
    # round 1: slot 2 bids rank 2 (self, 1.0; rank 3 also 1.0, lowest wins), slot 3 bids rank 2 too;
    #          rank 2 serves slot 2 (lowest slot), x = 1.
    # round 2: rank 2 is empty; both slots bid rank 3 (1.0); it serves slot 2, x = 1 -> slot 2 done.
    # round 3: slot 3 bids rank 0 (1/3, ties rank 1, lowest), x = 2, done.
    _, B = _two_node_B()
    n = np.zeros((4, 4), np.int32); n[:, 0] = [10, 10, 1, 1]
    a = O.auction(4, 4, 1, n, [-1, -1, 0, 0], [0, 0, 2, 2], B)
    assert a["X"][:, 2].tolist() == [0, 0, 1, 1] and a["X"][:, 3].tolist() == [2, 0, 0, 0]
    assert a["rounds"] == 3
    # with a steep price the second unit for slot 3 would come from the other cheap rank:
    # slot wanting 25 from ranks 0/1 (both 1/3 bonus from node 1, 10 tokens each) and 5 more at rank 2's node
    n[:, 0] = [10, 10, 0, 5]
    a = O.auction(4, 4, 1, n, [-1, -1, 0, -1], [0, 0, 25, 0], B, price_step=0.1)
    # round 1: rank 3 (intra, 1.0) gives 5; round 2: rank 0 gives 10; round 3: rank 1 (1/3) beats nobody else, gives 10
    assert a["X"][:, 2].tolist() == [10, 10, 0, 5] and a["rounds"] == 3


def test_auction_round_cap_leaves_residual():
    _, B = _two_node_B()
    n = np.zeros((4, 4), np.int32); n[:, 0] = [4, 0, 3, 3]
    a = O.auction(4, 4, 1, n, [-1, 0, -1, -1], [0, 5, 0, 0], B, max_rounds=1)
    assert a["rounds"] == 1 and a["residual"] == 1 and a["X"][:, 1].tolist() == [4, 0, 0, 0]


# ---------------------------------------------------------------------------- whole path invariants


@pytest.mark.parametrize("name,L,T", [("cfg1", 1, 4096), ("cfg2", 4, 16384), ("cfg3", 2, 32768), ("cfg4", 1, 65536)])
def test_schedule_constraints_on_synthetic_routing(name, L, T):
    cfg = W.get_config(name).replace(L=L, T=T)
    R, E, K = cfg.R, cfg.E, cfg.K
    topk = W.routing_topk(cfg).numpy()
    e2r = W.expert_to_rank(E, R, cfg.e2r_mode).numpy()
    C = W.cost_matrix(R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group).numpy()
    out = O.plan_layers(topk, R, E, K, e2r, C, cfg.eps, min(cfg.max_iters, 300), cfg.tol)
    tpr = T // R
    for l in range(L):
        n, el, rl = out["n"][l], out["expert_load"][l], out["rank_load"][l]
        mean, ex, sp = out["mean"][l], out["excess"][l], out["spare"][l]
        spill = O.spill(el, e2r, R, mean)
        se, stk, X = out["slot_expert"][l], out["slot_tokens"][l], out["X"][l]
        # Phase 2 constraints (Appendix A.3): per-expert spill, per-rank spare, K slots, never home, no duplicates
        assert ((se >= 0) == (stk > 0)).all()
        used = np.zeros(E, np.int64)
        for r in range(R):
            placed = [e for e in se[r] if e >= 0]
            assert len(set(placed)) == len(placed) and all(e2r[e] != r for e in placed)
            assert stk[r].sum() <= sp[r]
            for kap in range(K):
                if se[r, kap] >= 0:
                    used[se[r, kap]] += stk[r, kap]
        assert (used <= spill).all()
        assert stk.sum() <= min(spill.sum(), sp.sum())
        assert stk.sum() > 0                                      # the skewed routing does get balanced
        # Phase 3 constraints (Appendix A.4): column sums = A, per-(rank, expert) capacity
        assert (X.sum(0) == stk.ravel()).all()
        taken = np.zeros((R, E), np.int64)
        for s in range(R * K):
            if se.ravel()[s] >= 0:
                taken[:, se.ravel()[s]] += X[:, s]
            else:
                assert (X[:, s] == 0).all()
        assert (taken <= n).all()
        # reassignment: token conservation, counts equal X, earliest entries move
        new = out["new_idx"][l]
        assert new.shape == topk[l].shape
        src = np.repeat(np.arange(T) // tpr, cfg.k)
        flat_old, flat_new = topk[l].ravel(), new.ravel()
        moved = flat_new != flat_old
        assert (flat_new[moved] >= E).all() and (flat_new[~moved] < E).all()
        cnt = np.bincount(src[moved] * (R * K) + (flat_new[moved] - E), minlength=R * R * K).reshape(R, R * K)
        assert (cnt == X).all()
        assert (se.ravel()[flat_new[moved] - E] == flat_old[moved]).all()   # a moved entry lands on a replica of its own expert
        # earliest-first, lowest-slot-first: within each (source rank, expert) group the new targets, read in
        # flat order, are non-decreasing slots followed by the unmoved rest (pandas supplies the group ordinal)
        df = pd.DataFrame(dict(src=src, e=flat_old, new=flat_new))
        df["ord"] = df.groupby(["src", "e"]).cumcount()
        mv = df[df.new >= E]
        quota = taken
        assert (mv.ord.values < quota[mv.src.values, mv.e.values]).all()    # only the first quota entries move
        stay = df[df.new < E]
        assert (stay.ord.values >= quota[stay.src.values, stay.e.values]).all()
        key = mv.sort_values(["src", "e", "ord"])
        same = (key.src.values[1:] == key.src.values[:-1]) & (key.e.values[1:] == key.e.values[:-1])
        assert (key.new.values[1:][same] >= key.new.values[:-1][same]).all()
        # projected loads after the plan: imbalance does not get worse, here it improves
        after = rl.astype(np.int64).copy()
        for s in range(R * K):
            e = se.ravel()[s]
            if e >= 0:
                after[e2r[e]] -= stk.ravel()[s]; after[s // K] += stk.ravel()[s]
        assert after.max() < rl.max() and after.sum() == rl.sum()
        assert after.max() >= mean


def test_assign_hand_case():
    # R=2 (tokens 0-3 belong to rank 0, 4-7 to rank 1), k=1, E=2, K=1.  Slot 1 (rank 1) holds expert 0.
    # Rank 0 sends 2 of its expert-0 entries, rank 1 sends 1: the earliest ones move.
    topk = np.array([0, 1, 0, 0, 0, 0, 1, 0], np.int32).reshape(8, 1)
    X = np.array([[0, 2], [0, 1]], np.int32)
    new = O.assign(topk, 2, 2, 1, [-1, 0], X)
    assert new.ravel().tolist() == [3, 1, 3, 0, 3, 0, 1, 0]
    # two replicas of the same expert: lowest slot fills first
    X = np.array([[1, 2], [0, 0]], np.int32)
    new = O.assign(np.zeros((8, 1), np.int32), 2, 2, 1, [0, 0], X)
    assert new.ravel().tolist() == [2, 3, 3, 0, 0, 0, 0, 0]
    # out-of-range entries are copied through (tokens 2, 3 belong to rank 1, which sends one entry)
    new = O.assign(np.array([[5], [-3], [0], [0]], np.int32), 2, 2, 1, [-1, 0], np.array([[0, 0], [0, 1]], np.int32))
    assert new.ravel().tolist() == [5, -3, 3, 0]
