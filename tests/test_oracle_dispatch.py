"""Pins of the oracle's dispatch metadata (send counts, target counts, stable destination-sorted
permutation): a hand case, the defining properties checked directly, and a recomputation by a
different route (group ordinals with pandas)."""
import numpy as np
import pandas as pd

import oracle as O
import workloads as W


def test_dispatch_hand_case():
    # R=2, E=4 (experts 0,1 on rank 0; 2,3 on rank 1), K=1 -> slots 4 (rank 0), 5 (rank 1); T=4, k=2
    # source rank 0 owns entries [3, 5, 0, 3], source rank 1 owns [4, 1, 1, 2]
    new = np.array([[3, 5], [0, 3], [4, 1], [1, 2]], np.int32)
    d = O.dispatch(new, 2, 4, 1, [0, 0, 1, 1])
    # rank 0: destinations 1,1,0,1; sorted by (dest, target, order): 0@0 | 3(first) 3(second) 5 -> positions
    #   entry0 (3) -> 1, entry1 (5) -> 3, entry2 (0) -> 0, entry3 (3) -> 2
    # rank 1: targets 4 (rank 0), 1 (rank 0), 1 (rank 0), 2 (rank 1): order 1,1,4 | 2 ->
    #   entry0 (4) -> 2, entry1 (1) -> 0, entry2 (1) -> 1, entry3 (2) -> 3
    assert d["perm"].ravel().tolist() == [1, 3, 0, 2, 2, 0, 1, 3]
    assert d["send_counts"].tolist() == [[1, 3], [3, 1]]
    assert d["target_counts"].tolist() == [[1, 0, 0, 2, 0, 1], [0, 2, 1, 0, 1, 0]]
    assert d["bad"] == 0


def test_dispatch_undeliverable_indices_sort_last_in_order():
    new = np.array([[9, 1], [-3, 0]], np.int32)      # R=1: one segment [9, 1, -3, 0]; E=2, K=1 -> valid < 3
    d = O.dispatch(new, 1, 2, 1, [0, 0])
    assert d["perm"].ravel().tolist() == [2, 1, 3, 0]
    assert d["send_counts"].tolist() == [[2]] and d["bad"] == 2


def test_dispatch_properties_on_a_planned_layer():
    cfg = W.get_config("cfg1").replace(L=2, seed=91)
    tk = W.routing_topk(cfg).numpy()
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode).numpy()
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group).numpy()
    out = O.plan_layers(tk, cfg.R, cfg.E, cfg.K, e2r, C, cfg.eps, cfg.max_iters, cfg.tol)
    B = O.default_preference(C)
    seg = cfg.T // cfg.R * cfg.k
    for l in range(cfg.L):
        new = out["new_idx"][l]
        d = O.dispatch(new, cfg.R, cfg.E, cfg.K, e2r)
        flat = new.reshape(cfg.R, seg); perm = d["perm"].reshape(cfg.R, seg)
        dest = np.where(flat < cfg.E, e2r[np.minimum(flat, cfg.E - 1)], (flat - cfg.E) // cfg.K)
        for r in range(cfg.R):
            assert sorted(perm[r].tolist()) == list(range(seg))                  # a permutation
            buf_t = np.empty(seg, np.int64); buf_d = np.empty(seg, np.int64); buf_i = np.empty(seg, np.int64)
            buf_t[perm[r]] = flat[r]; buf_d[perm[r]] = dest[r]; buf_i[perm[r]] = np.arange(seg)
            assert (np.diff(buf_d) >= 0).all()                                   # grouped by destination rank
            same_d = np.diff(buf_d) == 0
            assert (np.diff(buf_t)[same_d] >= 0).all()                           # then by target
            same_t = same_d & (np.diff(buf_t) == 0)
            assert (np.diff(buf_i)[same_t] > 0).all()                            # stable
            # a different route to the same positions: rank of the key plus ordinal within the key group
            key = dest[r] * (cfg.E + cfg.S) + flat[r]
            ordinal = pd.Series(key).groupby(key).cumcount().to_numpy()
            uniq, cnt = np.unique(key, return_counts=True)
            start = dict(zip(uniq.tolist(), (np.cumsum(cnt) - cnt).tolist()))
            assert (perm[r] == np.array([start[kk] for kk in key.tolist()]) + ordinal).all()
        assert (d["send_counts"].sum(1) == seg).all()
        # what each rank receives is its projected load of the dispatch report
        rep = O.report(cfg.R, cfg.E, cfg.K, e2r, C, B, out["expert_load"][l], out["rank_load"][l],
                       out["slot_expert"][l], out["X"][l])
        assert (d["send_counts"].sum(0) == rep["load_after"]).all()
        # guest-slot columns of the target counts are the auction's X
        assert (d["target_counts"][:, cfg.E:] == out["X"][l]).all()
