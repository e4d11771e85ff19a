"""Algorithm-level ablation on synthetic imbalanced routing (the paper's Ablation Study, Table 2): run the planner
with the Phase-1 flow hint and the Phase-2 topology term switched off / on and print, per setting, the final
imbalance, the intra-/inter-node transfer counts and the weighted cost at 1:lambda, mean +/- std over the layers
of the workload that sit at the chosen imbalance level.  Everything is computed on the GPU (taot_plan, taot_report).

    python -m paper_2608_03676_b200.ablation --workload ladder32 --level 4
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

import workloads as W
from . import ABLATE_HINT, ABLATE_TOPOLOGY, Planner


def run(workload: str = "ladder32", level: int = -1, lam: float = 3.0):
    cfg = W.get_config(workload)
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode)
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group)
    topk = W.routing_topk(cfg, device="cuda")
    nlev = max(1, len(cfg.rank_fracs))
    layers = [l for l in range(cfg.L) if level < 0 or l % nlev == level]
    rows = []
    for hint, topo in ((False, False), (False, True), (True, False), (True, True)):
        flags = (0 if hint else ABLATE_HINT) | (0 if topo else ABLATE_TOPOLOGY)
        pl = Planner(L=cfg.L, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r, C=C, eps=cfg.eps,
                     max_iters=cfg.max_iters, tol=cfg.tol, ablation=flags)
        out = pl.plan(topk)
        rep = pl.report(out["expert_load"], out["rank_load"], out["slot_expert"], out["X"], lam)
        torch.cuda.synchronize()
        sel = lambda key: np.asarray(rep[key])[layers].astype(np.float64)
        rows.append(dict(hint=hint, topology=topo, layers=len(layers),
                         initial_imbalance_pct=[float(100 * sel("rho_before").mean()), float(100 * sel("rho_before").std())],
                         final_imbalance_pct=[float(100 * sel("rho_after").mean()), float(100 * sel("rho_after").std())],
                         intra=[float(sel("intra").mean()), float(sel("intra").std())],
                         inter=[float(sel("inter").mean()), float(sel("inter").std())],
                         weighted_cost=[float(sel("cost_ratio").mean()), float(sel("cost_ratio").std())]))
        pl.close()
    return rows


def main():
    ap = argparse.ArgumentParser(description=__doc__)
    ap.add_argument("--workload", default="ladder32")
    ap.add_argument("--level", type=int, default=-1, help="index into the workload's imbalance levels (-1: all layers)")
    ap.add_argument("--lambda", dest="lam", type=float, default=3.0)
    ap.add_argument("--json", action="store_true")
    a = ap.parse_args()
    rows = run(a.workload, a.level, a.lam)
    if a.json:
        print(json.dumps(rows))
        return
    print(f"{'hint':>5} {'topo':>5} {'initial %':>16} {'final imbalance %':>20} {'intra':>14} {'inter':>14} {'weighted cost':>16}")
    pm = lambda v: f"{v[0]:.2f} +/- {v[1]:.2f}"
    for r in rows:
        print(f"{'on' if r['hint'] else 'off':>5} {'on' if r['topology'] else 'off':>5} {pm(r['initial_imbalance_pct']):>16} "
              f"{pm(r['final_imbalance_pct']):>20} {pm(r['intra']):>14} {pm(r['inter']):>14} {pm(r['weighted_cost']):>16}")


if __name__ == "__main__":
    main()
