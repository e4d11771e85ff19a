"""Shared helpers of the GPU parity tests: build a planner for a workload config, run the oracle
stage by stage on the same arrays, and the comparison rules (bit-exact integers; Sinkhorn within
1e-4 relative per entry and 1e-5 of total mass on the marginals)."""
from __future__ import annotations

import numpy as np
import torch

import oracle as O
import workloads as W

REL_TOL = 1e-4          # per-entry relative error of the plan
MASS_TOL = 1e-5         # marginal violation as a fraction of total mass
STOP_BAND = 5e-7        # band around tol inside which the fp32 stopping decision may differ


def topology(cfg):
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode)
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group)
    return e2r, C


def make_planner(cfg, **over):
    import paper_2608_03676_b200 as P
    e2r, C = topology(cfg)
    kw = dict(L=cfg.L, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r, C=C, eps=cfg.eps,
              max_iters=cfg.max_iters, tol=cfg.tol)
    kw.update(over)
    return P.Planner(**kw)


def check_sinkhorn_problem(s, d, C, eps, gpu_plan, gpu_iters, gpu_err, max_iters, tol, check_every=1,
                           eps0=1e-8, err_band=STOP_BAND):
    """Replay the oracle for exactly the iteration count the GPU reports and compare.  err_band: how far the row
    error the GPU reports may be from the oracle's (the plan's own marginals are always held to MASS_TOL)."""
    R = len(s)
    ref = O.sinkhorn(s, d, C, eps, max(int(gpu_iters), 1) if gpu_iters > 0 else 1, 0.0, 1, eps0,
                     history=(tol > 0 and gpu_iters > 0))
    s64 = s.astype(np.float64); d64 = d.astype(np.float64)
    gamma = min(1.0, d64.sum() / max(s64.sum(), eps0))
    st = gamma * s64
    total = st.sum()
    gp = gpu_plan.astype(np.float64)
    if gpu_iters == 0:
        assert total == 0 or d64.sum() == 0
        assert (gp == 0).all()
        return dict(max_rel=0.0)
    T = ref["plan"]
    tau = 1e-7 * total / (R * R)
    rel = np.abs(gp - T) / np.maximum(T, tau)
    assert rel.max() <= REL_TOL, f"plan max rel err {rel.max():.3e}"
    assert (gp >= 0).all() and np.isfinite(gp).all()
    assert (gp[st == 0, :] == 0).all() and (gp[:, d64 == 0] == 0).all()
    col_viol = np.abs(gp.sum(0) - d64).sum()
    assert col_viol <= MASS_TOL * total, f"column violation {col_viol / total:.3e}"
    row_viol_gpu = np.abs(gp.sum(1) - st).sum()
    row_viol_ref = np.abs(T.sum(1) - st).sum()
    assert abs(row_viol_gpu - row_viol_ref) <= MASS_TOL * total
    assert abs(float(gpu_err) - ref["row_err"]) <= max(err_band, 1e-3 * ref["row_err"])
    if tol > 0:
        h = ref["err_hist"]
        n = int(gpu_iters)
        assert n % check_every == 0 or n == max_iters
        if n < max_iters:
            assert h[n - 1] <= tol + STOP_BAND                       # it did have reason to stop
        prev = n - check_every
        if prev >= 1:
            assert h[prev - 1] > tol - STOP_BAND                     # and none to stop earlier
        if n == max_iters and h[n - 1] > tol + STOP_BAND:
            pass                                                     # capped: flagged via info
        else:
            assert row_viol_gpu <= (tol + STOP_BAND + MASS_TOL) * total
    return dict(max_rel=float(rel.max()))


def oracle_schedule_layer(cfg, e2r, B, n, el, rl, plan32, price_step=0.1, auction_max_rounds=0, eps0=1e-8):
    """Phases 2 and 3 of the oracle for one layer, fed the given fp32 plan."""
    mean, ex, sp = O.excess_spare(rl[None])
    spill = O.spill(el, e2r, cfg.R, mean[0])
    m = O.match(cfg.R, cfg.E, cfg.K, e2r, mean[0], ex[0], spill, sp[0], B, plan32, eps0)
    a = O.auction(cfg.R, cfg.E, cfg.K, n, m["slot_expert"], m["slot_tokens"], B, price_step, auction_max_rounds)
    return m, a


def cpu(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()
