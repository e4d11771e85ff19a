"""The five benchmark configurations, as plain data.

Shapes follow the planner's problem statement (R expert-parallel ranks, E experts, K guest
slots per rank, router top-k) and the workload description: Zipf-skewed routing over a
seeded expert permutation, a tiered rank-to-rank communication cost (0 self / intra-node /
[rail group] / cross-node) and an entropic regulariser given as a fraction of max(C).
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Optional, Tuple

BASE_SEED = 20260803


@dataclass(frozen=True)
class PlannerConfig:
    name: str
    L: int                      # independent problems: MoE layers x micro-batches
    R: int                      # EP ranks
    E: int                      # experts
    K: int                      # guest slots per rank
    k: int                      # router top-k
    T: int                      # tokens per layer (T % R == 0; rank r owns tokens [r*T/R, (r+1)*T/R))
    gpus_per_node: int
    tiers: Tuple[float, ...]    # (self, intra-node, cross-node) or (self, intra, rail-group, other)
    nodes_per_group: Optional[int] = None
    e2r_mode: str = "contiguous"   # "contiguous": e // (E/R);  "stride2": e -> 2e (odd ranks host nothing)
    zipf: Tuple[float, float] = (1.0, 1.0)   # per-layer exponent ~ U[lo, hi]
    hot_frac: float = 0.0       # fraction of tokens forced onto one random expert per layer
    rank_fracs: Tuple[float, ...] = ()   # if set: layer l sends fraction rank_fracs[l % len] of its tokens to
                                         # the experts of one random rank and the rest to uniformly random experts
    eps_frac: float = 0.05      # eps = eps_frac * max(C)
    max_iters: int = 200
    tol: float = 0.0            # <= 0: exactly max_iters iterations
    seed: int = BASE_SEED

    @property
    def tokens_per_rank(self) -> int:
        return self.T // self.R

    @property
    def S(self) -> int:
        return self.R * self.K

    @property
    def eps(self) -> float:
        return self.eps_frac * max(self.tiers)

    def replace(self, **kw) -> "PlannerConfig":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "cfg1": PlannerConfig("cfg1", L=1, R=8, E=32, K=2, k=2, T=4096, gpus_per_node=4,
                          tiers=(0.0, 1.0, 8.0), zipf=(1.2, 1.2), eps_frac=0.05,
                          max_iters=200, tol=0.0),
    "cfg2": PlannerConfig("cfg2", L=24, R=16, E=64, K=2, k=8, T=16384, gpus_per_node=8,
                          tiers=(0.0, 1.0, 10.0), zipf=(1.0, 1.0), eps_frac=0.02,
                          max_iters=1000, tol=1e-6),
    "cfg3": PlannerConfig("cfg3", L=58, R=64, E=256, K=2, k=8, T=524288, gpus_per_node=8,
                          tiers=(0.0, 1.0, 12.0), zipf=(0.8, 1.4), hot_frac=0.05,
                          eps_frac=0.01, max_iters=1000, tol=1e-6),
    "cfg4": PlannerConfig("cfg4", L=48, R=256, E=128, K=1, k=8, T=1048576, gpus_per_node=8,
                          tiers=(0.0, 1.0, 6.0, 16.0), nodes_per_group=4, e2r_mode="stride2",
                          zipf=(0.6, 1.6), eps_frac=0.005, max_iters=1000, tol=1e-6),
    # Imbalance built as in the paper's sensitivity study: 30/50/70/90 % of the tokens go to one rank, the
    # rest at random; EP32, E=256, K=2, cost 1 intra-node / lambda=3 cross-node, eps = lambda.  3 seeds per level.
    "llep32": PlannerConfig("llep32", L=12, R=32, E=256, K=2, k=8, T=65536, gpus_per_node=8,
                            tiers=(0.0, 1.0, 3.0), eps_frac=1.0, max_iters=1000, tol=1e-6,
                            rank_fracs=(0.3, 0.5, 0.7, 0.9)),
    # The initial-imbalance ladder of the balance-quality study: rho_0 in {10,20,30,50,70} %, reached by sending
    # the fraction rho_0/(R-1) of the tokens to one rank; EP16 and EP32, 3 seeds per level.
    "ladder16": PlannerConfig("ladder16", L=15, R=16, E=256, K=2, k=8, T=32768, gpus_per_node=8,
                              tiers=(0.0, 1.0, 3.0), eps_frac=1.0, max_iters=1000, tol=1e-6,
                              rank_fracs=tuple(x / 15.0 for x in (0.1, 0.2, 0.3, 0.5, 0.7))),
    "ladder32": PlannerConfig("ladder32", L=15, R=32, E=256, K=2, k=8, T=65536, gpus_per_node=8,
                              tiers=(0.0, 1.0, 3.0), eps_frac=1.0, max_iters=1000, tol=1e-6,
                              rank_fracs=tuple(x / 31.0 for x in (0.1, 0.2, 0.3, 0.5, 0.7))),
}


def get_config(name: str) -> PlannerConfig:
    return CONFIGS[name]


def sweep_cells(batches=(1, 64, 1024, 4096), ranks=(8, 16, 64, 256, 1024), eps_fracs=(0.1, 0.01)):
    """Config 5: Sinkhorn-only scaling sweep; each cell is (B, R, eps_frac), 500 fixed iterations,
    3-tier cost with 8 GPUs per node and 4 nodes per rail group."""
    return [(B, R, f) for R in ranks for B in batches for f in eps_fracs]


SWEEP_TIERS = (0.0, 1.0, 6.0, 16.0)
SWEEP_ITERS = 500
SWEEP_LOAD_PER_RANK = 32768
SWEEP_ZIPF = 1.2
