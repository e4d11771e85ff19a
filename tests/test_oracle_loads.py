"""Pins for the oracle's load collection, excess/spare and spill (Appendix A.1, A.3)."""
import json
import os

import numpy as np
import pytest

import oracle as O
import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_histogram_matches_bincount():
    cfg = W.get_config("cfg2").replace(L=3, T=4096)
    topk = W.routing_topk(cfg).numpy()
    e2r = W.expert_to_rank(cfg.E, cfg.R).numpy()
    n, el, rl, bad = O.histogram(topk, cfg.R, cfg.E, e2r)
    tpr = cfg.T // cfg.R
    for l in range(cfg.L):
        src = np.repeat(np.arange(cfg.T) // tpr, cfg.k)
        joint = np.bincount(src * cfg.E + topk[l].ravel(), minlength=cfg.R * cfg.E).reshape(cfg.R, cfg.E)
        assert (n[l] == joint).all()
        assert (el[l] == np.bincount(topk[l].ravel(), minlength=cfg.E)).all()
        assert (rl[l] == np.bincount(e2r, weights=el[l], minlength=cfg.R).astype(np.int64)).all()
    assert (bad == 0).all()
    assert n.sum() == cfg.L * cfg.T * cfg.k


def test_histogram_counts_and_skips_bad_indices():
    topk = np.array([[[0, 1], [7, -1], [2, 2], [1, 8]]], np.int32)      # L=1, T=4, k=2, E=8, R=2
    e2r = np.arange(8, dtype=np.int32) // 4
    n, el, rl, bad = O.histogram(topk, 2, 8, e2r)
    assert bad.tolist() == [2]
    assert n[0, 0].tolist() == [1, 1, 0, 0, 0, 0, 0, 1]
    assert n[0, 1].tolist() == [0, 1, 2, 0, 0, 0, 0, 0]
    assert rl[0].tolist() == [5, 1]


def test_excess_spare_definition_and_balance():
    rl = np.array([[28, 8, 24, 4], [10, 10, 10, 11], [0, 0, 0, 0]], np.int32)
    mean, ex, sp = O.excess_spare(rl)
    assert mean.tolist() == [16, 10, 0]                                  # integer (floor) mean
    assert ex[0].tolist() == [12, 0, 8, 0] and sp[0].tolist() == [0, 8, 0, 12]
    assert ex[1].tolist() == [0, 0, 0, 1] and sp[1].tolist() == [0, 0, 0, 0]
    # sum(excess) - sum(spare) == total mod R
    assert (ex.sum(1) - sp.sum(1)).tolist() == [0, 41 % 4, 0]
    assert ((ex > 0) & (sp > 0)).sum() == 0                              # hot and cold sets are disjoint


def test_spill_identities_random():
    rng = np.random.default_rng(0)
    for _ in range(50):
        R = int(rng.integers(2, 9)); per = int(rng.integers(1, 6)); E = R * per
        e2r = np.repeat(np.arange(R), per).astype(np.int32)
        el = rng.integers(0, 100, size=E).astype(np.int32)
        rl = np.bincount(e2r, weights=el, minlength=R).astype(np.int32)[None]
        mean, ex, sp = O.excess_spare(rl)
        spill = O.spill(el, e2r, R, mean[0])
        assert (spill >= 0).all() and (spill <= el).all()
        per_rank = np.bincount(e2r, weights=spill, minlength=R).astype(np.int64)
        assert (per_rank == ex[0]).all()                                 # sum over a rank's experts = its excess
        for r in range(R):
            mine = np.where(e2r == r)[0]
            # the lightest experts carry no spill: only a suffix of the load-sorted order does
            order = mine[np.lexsort((mine, el[mine]))]
            s = spill[order]
            nz = np.nonzero(s)[0]
            if len(nz):
                assert (s[nz[0] + 1:] == el[order][nz[0] + 1:]).all()    # after the first spilling expert, all of it spills


def test_spill_hand_case():
    g = json.load(open(os.path.join(GOLD, "w1_hand_trace.json")))
    spill = O.spill(np.array(g["expert_load"], np.int32), np.array(g["e2r"], np.int32), g["R"], g["mean"])
    assert spill.tolist() == g["spill"]
    # sorted loads (3, 9, 20) on one rank against mean 10: sigma = 0, 2, 22 -> spill 0, 2, 20
    spill = O.spill(np.array([20, 3, 9], np.int32), np.zeros(3, np.int32), 1, 10)
    assert spill.tolist() == [20, 0, 2]
