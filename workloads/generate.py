"""Counter-based, device-agnostic generators for the planner's synthetic inputs.

Everything random is a pure function of (seed, stream, counter) through a 64-bit integer
mixer, so any slice of any tensor can be regenerated independently and a CPU run and a CUDA
run follow the same recipe.  (The routing keys go through a float64 log; the two devices'
log may differ in the last bit, so tests always hand *one* generated array to both sides.)
"""
from __future__ import annotations

import math
from typing import Optional, Sequence

import torch

from .configs import (PlannerConfig, SWEEP_LOAD_PER_RANK, SWEEP_ZIPF)

_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit constant as the signed value torch.int64 stores."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 lanes (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    """The splitmix64 finaliser on int64 lanes (wrap-around multiply)."""
    z = z + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _hash(seed: int, stream: int, counter: torch.Tensor) -> torch.Tensor:
    key = _s64((seed * 0x2545F4914F6CDD1D + stream * 0xD6E8FEB86659FD93) & _MASK64)
    return _mix(_mix(counter) ^ key)


def uniform01(seed: int, stream: int, counter: torch.Tensor) -> torch.Tensor:
    """float64 uniforms in the open interval (0, 1), one per counter value."""
    h = _lsr(_hash(seed, stream, counter), 11)            # 53 random bits
    return (h.to(torch.float64) + 0.5) * (2.0 ** -53)


# ----------------------------------------------------------------------------------------
# topology


def cost_matrix(R: int, gpus_per_node: int, tiers: Sequence[float],
                nodes_per_group: Optional[int] = None, device="cpu") -> torch.Tensor:
    """Rank-by-rank communication cost, float32 [R, R].

    tiers = (self, intra-node, cross-node) or (self, intra-node, same rail group, otherwise).
    Ranks are numbered node-major: node = r // gpus_per_node, group = node // nodes_per_group.
    """
    r = torch.arange(R, device=device)
    node = r // gpus_per_node
    same_node = node[:, None] == node[None, :]
    if len(tiers) == 3:
        C = torch.full((R, R), float(tiers[2]), dtype=torch.float32, device=device)
        C[same_node] = float(tiers[1])
    else:
        assert nodes_per_group is not None
        grp = node // nodes_per_group
        same_grp = grp[:, None] == grp[None, :]
        C = torch.full((R, R), float(tiers[3]), dtype=torch.float32, device=device)
        C[same_grp] = float(tiers[2])
        C[same_node] = float(tiers[1])
    C[r, r] = float(tiers[0])
    return C


def expert_to_rank(E: int, R: int, mode: str = "contiguous", device="cpu") -> torch.Tensor:
    """Home rank of every expert, int32 [E]."""
    e = torch.arange(E, device=device)
    if mode == "contiguous":
        assert E % R == 0
        return (e // (E // R)).to(torch.int32)
    if mode == "stride2":
        assert 2 * E <= R
        return (2 * e).to(torch.int32)
    raise ValueError(mode)


# ----------------------------------------------------------------------------------------
# routing tables


def zipf_exponents(cfg: PlannerConfig, device="cpu") -> torch.Tensor:
    lo, hi = cfg.zipf
    u = uniform01(cfg.seed, 1, torch.arange(cfg.L, dtype=torch.int64, device=device))
    return lo + (hi - lo) * u


def _layer_log_popularity(cfg: PlannerConfig, layer: int, device) -> torch.Tensor:
    """log p_e for one layer: Zipf over a seeded permutation of the experts."""
    E = cfg.E
    lo, hi = cfg.zipf
    u = uniform01(cfg.seed, 1, torch.tensor([layer], dtype=torch.int64, device=device))
    s = lo + (hi - lo) * float(u[0])
    order_keys = _hash(cfg.seed, 2, layer * E + torch.arange(E, dtype=torch.int64, device=device))
    rank_of_expert = torch.empty(E, dtype=torch.int64, device=device)
    rank_of_expert[torch.argsort(order_keys, stable=True)] = torch.arange(E, device=device)
    logp = -s * torch.log(rank_of_expert.to(torch.float64) + 1.0)
    return logp - torch.logsumexp(logp, 0)


def routing_topk(cfg: PlannerConfig, device="cpu", layers: Optional[Sequence[int]] = None,
                 max_chunk_elems: int = 1 << 23) -> torch.Tensor:
    """Router output topk_idx, int32 [L, T, k]: k distinct experts per token.

    Sampling without replacement from the layer's popularity uses the Gumbel-top-k
    construction (perturb log p_e with an independent Gumbel per (token, expert), keep the
    k largest, emit in descending-key order).  With cfg.hot_frac > 0, that fraction of
    tokens has its last choice replaced by one per-layer hot expert unless already chosen.
    """
    L, T, E, k = cfg.L, cfg.T, cfg.E, cfg.k
    layers = list(range(L)) if layers is None else list(layers)
    out = torch.empty((len(layers), T, k), dtype=torch.int32, device=device)
    chunk = max(1, min(T, max_chunk_elems // E))
    e_ids = torch.arange(E, dtype=torch.int64, device=device)
    if cfg.rank_fracs:
        return _routing_one_hot_rank(cfg, device, layers, out, chunk, e_ids)
    for li, layer in enumerate(layers):
        logp = _layer_log_popularity(cfg, layer, device)
        if cfg.hot_frac > 0:
            uh = uniform01(cfg.seed, 4, torch.tensor([layer], dtype=torch.int64, device=device))
            hot = min(E - 1, int(float(uh[0]) * E))
        for t0 in range(0, T, chunk):
            t1 = min(T, t0 + chunk)
            tok = torch.arange(t0, t1, dtype=torch.int64, device=device)
            ctr = ((layer * T + tok)[:, None]) * E + e_ids[None, :]
            u = uniform01(cfg.seed, 3, ctr)
            keys = logp[None, :] - torch.log(-torch.log(u))
            idx = torch.topk(keys, k, dim=1, largest=True, sorted=True).indices
            if cfg.hot_frac > 0:
                ut = uniform01(cfg.seed, 5, layer * T + tok)
                force = (ut < cfg.hot_frac) & ~(idx == hot).any(dim=1)
                idx[force, k - 1] = hot
            out[li, t0:t1] = idx.to(torch.int32)
    return out


def _routing_one_hot_rank(cfg, device, layers, out, chunk, e_ids):
    """Routing with a fraction of the tokens sent to one rank: in layer l a token is "hot" with probability
    rank_fracs[l % len]; a hot token's k choices are k distinct experts of the layer's hot rank (seeded), any
    other token's are k distinct uniformly random experts.  Needs k <= experts per rank."""
    T, E, k, R = cfg.T, cfg.E, cfg.k, cfg.R
    home = expert_to_rank(E, R, cfg.e2r_mode, device=device).to(torch.int64)
    for li, layer in enumerate(layers):
        f = cfg.rank_fracs[layer % len(cfg.rank_fracs)]
        uh = uniform01(cfg.seed, 7, torch.tensor([layer], dtype=torch.int64, device=device))
        hot_rank = min(R - 1, int(float(uh[0]) * R))
        on_hot = home == hot_rank
        assert int(on_hot.sum()) >= k, "the hot rank must host at least k experts"
        bar = torch.where(on_hot, 0.0, -float("inf")).to(torch.float64)
        for t0 in range(0, T, chunk):
            t1 = min(T, t0 + chunk)
            tok = torch.arange(t0, t1, dtype=torch.int64, device=device)
            ctr = ((layer * T + tok)[:, None]) * E + e_ids[None, :]
            keys = -torch.log(-torch.log(uniform01(cfg.seed, 3, ctr)))
            hot_tok = uniform01(cfg.seed, 8, layer * T + tok) < f
            keys = torch.where(hot_tok[:, None], keys + bar[None, :], keys)
            out[li, t0:t1] = torch.topk(keys, k, dim=1, largest=True, sorted=True).indices.to(torch.int32)
    return out


# ----------------------------------------------------------------------------------------
# Sinkhorn-only sweep (config 5): per-problem rank loads


def sweep_rank_loads(B: int, R: int, seed: int, device="cpu",
                     load_per_rank: int = SWEEP_LOAD_PER_RANK, zipf: float = SWEEP_ZIPF) -> torch.Tensor:
    """Integer rank loads, int32 [B, R], each row summing to exactly load_per_rank * R.

    Row b: p_r proportional to (pi_b(r) + 1)^(-zipf) for a seeded permutation pi_b of the
    ranks; loads are load_per_rank * R * p rounded by the largest-remainder rule (floors,
    then one extra unit to the largest fractional parts, ties to the lower rank).
    """
    ctr = torch.arange(B * R, dtype=torch.int64, device=device).reshape(B, R)
    keys = _hash(seed, 6, ctr)
    pos = torch.empty((B, R), dtype=torch.int64, device=device)
    order = torch.argsort(keys, dim=1, stable=True)
    pos.scatter_(1, order, torch.arange(R, device=device).expand(B, R).contiguous())
    w = (pos.to(torch.float64) + 1.0) ** (-zipf)
    p = w / w.sum(dim=1, keepdim=True)
    total = load_per_rank * R
    x = p * total
    base = torch.floor(x)
    rem = (total - base.sum(dim=1)).to(torch.int64)              # units still to hand out, per row
    frac = x - base
    by_frac = torch.argsort(-frac, dim=1, stable=True)
    rank_in_frac = torch.empty_like(by_frac)
    rank_in_frac.scatter_(1, by_frac, torch.arange(R, device=device).expand(B, R).contiguous())
    loads = base.to(torch.int64) + (rank_in_frac < rem[:, None]).to(torch.int64)
    assert bool((loads.sum(dim=1) == total).all())
    return loads.to(torch.int32)
