"""The synthetic input generators: determinism, shapes and the statistical structure they promise."""
import numpy as np
import torch

import workloads as W


def test_routing_is_deterministic_and_distinct():
    cfg = W.get_config("cfg1")
    a = W.routing_topk(cfg)
    b = W.routing_topk(cfg)
    assert a.dtype == torch.int32 and tuple(a.shape) == (cfg.L, cfg.T, cfg.k)
    assert torch.equal(a, b)
    s = torch.sort(a, dim=-1).values
    assert int((s[..., 1:] == s[..., :-1]).sum()) == 0          # k distinct experts per token
    assert int(a.min()) >= 0 and int(a.max()) < cfg.E
    c = W.routing_topk(cfg.replace(seed=cfg.seed + 1))
    assert not torch.equal(a, c)


def test_routing_layers_can_be_regenerated_independently():
    cfg = W.get_config("cfg2").replace(L=3, T=2048)
    full = W.routing_topk(cfg)
    only2 = W.routing_topk(cfg, layers=[2])
    assert torch.equal(full[2], only2[0])
    chunked = W.routing_topk(cfg, max_chunk_elems=64 * 100)     # chunk boundaries must not matter
    assert torch.equal(full, chunked)


def test_routing_is_zipf_skewed():
    cfg = W.get_config("cfg2").replace(L=1, T=16384)
    t = W.routing_topk(cfg).numpy().ravel()
    counts = np.sort(np.bincount(t, minlength=cfg.E))[::-1].astype(float)
    assert counts[0] > 4 * counts[cfg.E // 2]                   # head much heavier than the middle
    assert counts.sum() == cfg.T * cfg.k


def test_hot_expert_fraction():
    cfg = W.get_config("cfg3").replace(L=1, T=32768, zipf=(0.0, 0.0))
    t = W.routing_topk(cfg).numpy()
    counts = np.bincount(t.ravel(), minlength=cfg.E)
    hot = int(np.argmax(counts))
    base = cfg.T * cfg.k / cfg.E
    # uniform popularity: every expert gets ~T*k/E; the hot one gets ~5% of the tokens on top
    assert counts[hot] > base + 0.03 * cfg.T
    assert counts[hot] < base + 0.07 * cfg.T


def test_cost_matrix_tiers():
    C = W.cost_matrix(64, 8, (0.0, 1.0, 6.0, 16.0), 4).numpy()
    assert C.dtype == np.float32 and C.shape == (64, 64)
    assert (np.diag(C) == 0).all()
    assert C[0, 7] == 1 and C[0, 8] == 6 and C[0, 31] == 6 and C[0, 32] == 16
    assert (C == C.T).all()
    C3 = W.cost_matrix(8, 4, (0.0, 1.0, 8.0)).numpy()
    assert C3[0, 3] == 1 and C3[0, 4] == 8


def test_expert_to_rank():
    assert W.expert_to_rank(32, 8).tolist() == [e // 4 for e in range(32)]
    assert W.expert_to_rank(4, 8, "stride2").tolist() == [0, 2, 4, 6]


def test_sweep_loads_sum_exactly():
    l = W.sweep_rank_loads(5, 64, seed=3)
    assert l.dtype == torch.int32 and tuple(l.shape) == (5, 64)
    assert (l.sum(dim=1) == 32768 * 64).all()
    srt = torch.sort(l.double(), dim=1, descending=True).values
    assert torch.allclose(srt[0], srt[1])                       # same Zipf profile, permuted
    assert not torch.equal(l[0], l[1])
    ratio = float(srt[0, 0] / srt[0, 1])
    assert abs(ratio - 2 ** 1.2) < 0.01


def test_bench_recognises_the_tiered_costs_of_the_workloads():
    """bench.py decides from the cost matrix which Sinkhorn kernel the library takes (to count its work): the costs
    of config 4 and of the sweep from 256 ranks up are pure tier costs, smaller ones and perturbed ones are not."""
    import importlib.util
    import os
    import torch
    import workloads as W
    from workloads.configs import SWEEP_TIERS
    spec = importlib.util.spec_from_file_location("bench_mod", os.path.join(os.path.dirname(__file__), "..", "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    for R in (256, 512, 1024):
        assert bench.tiered_sums(W.cost_matrix(R, 8, SWEEP_TIERS, 4), 1)
    assert not bench.tiered_sums(W.cost_matrix(64, 8, SWEEP_TIERS, 4), 64)
    cfg = W.get_config("cfg4")
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group)
    assert bench.tiered_sums(C, cfg.L)
    C2 = C.clone(); C2[3, 77] += 1.0
    assert not bench.tiered_sums(C2, cfg.L)
    two_tier = W.cost_matrix(256, 8, (0.0, 1.0, 12.0), None)          # node / cross-node only: still a tier cost
    assert bench.tiered_sums(two_tier, 8)
    assert bench.tiered_fma_per_iteration(256) == 2 * (4 * 256 + 64 + 1)
