"""Text rendering of the per-layer dispatch report (Appendix B.3: four parts).  Formatting only: every number
printed here was computed on the GPU by `taot_report` (or is an input of it)."""
from __future__ import annotations

from typing import Dict, List

KIND = {0: "-", 1: "intra", 2: "inter", 3: "home"}


def _np(x):
    return x.detach().cpu().numpy() if hasattr(x, "detach") else x


def format_layer(rep: Dict[str, object], layer: int, rank_load, expert_load, slot_expert, e2r, K: int,
                 max_rows: int = 16) -> str:
    """One layer of `Planner.report(...)` as text.  rank_load [L,R], expert_load [L,E], slot_expert [L,R,K]
    are the planner outputs the report was computed from; e2r [E] is the home-rank map."""
    rl = _np(rank_load)[layer]; el = _np(expert_load)[layer]
    se = _np(slot_expert)[layer].reshape(-1); e2r = _np(e2r)
    spill = _np(rep["spill"])[layer]; after = _np(rep["load_after"])[layer]
    moved = _np(rep["slot_moved"])[layer]; kind = _np(rep["slot_kind"])[layer]
    g = lambda name: rep[name][layer]
    mean = int(g("mean_load"))
    out: List[str] = [f"== layer {layer} =="]
    out.append(f"(1) load before: total {int(g('total_load'))}, mean {mean}, max {int(g('max_before'))}, "
               f"min {int(g('min_before'))}; {int(g('hot_ranks'))} hot / {int(g('cold_ranks'))} cold ranks, "
               f"{int(g('hot_experts'))} hot experts")
    hot_r = [r for r in range(len(rl)) if rl[r] > mean]
    out.append("    hot ranks: " + ", ".join(f"r{r}={int(rl[r])}" for r in hot_r[:max_rows]) +
               (" ..." if len(hot_r) > max_rows else ""))
    hot_e = [e for e in range(len(el)) if spill[e] > 0]
    out.append("    hot experts (load, spill): " +
               ", ".join(f"e{e}@r{int(e2r[e])}=({int(el[e])},{int(spill[e])})" for e in hot_e[:max_rows]) +
               (" ..." if len(hot_e) > max_rows else ""))
    out.append("(2) cloning plan:")
    shown = 0
    for s in range(len(se)):
        if kind[s] == 0:
            continue
        if shown < max_rows:
            e = int(se[s])
            out.append(f"    e{e} (home r{int(e2r[e])}) -> slot {s} on r{s // K}: {KIND[int(kind[s])]}, "
                       f"{int(moved[s])} tokens")
        shown += 1
    if shown > max_rows:
        out.append(f"    ... {shown - max_rows} more")
    out.append(f"    copies: {int(g('clones'))} ({int(g('intra'))} intra-node, {int(g('inter'))} inter-node, "
               f"{int(g('same_rank'))} on the home rank); weighted cost {g('cost_ratio'):.2f} (1:lambda), "
               f"{g('cost_C'):.2f} (by C)")
    out.append(f"(3) projected load: max {int(g('max_after'))}, min {int(g('min_after'))}; " +
               ", ".join(f"r{r}={int(after[r])}" for r in range(min(len(after), max_rows))) +
               (" ..." if len(after) > max_rows else ""))
    out.append(f"(4) imbalance {100 * g('rho_before'):.2f}% -> {100 * g('rho_after'):.2f}% "
               f"(largest deviation {100 * g('dev_before'):.2f}% -> {100 * g('dev_after'):.2f}%), "
               f"peak load -{100 * g('peak_reduction'):.2f}%, {100 * g('frac_rerouted'):.2f}% of tokens rerouted")
    return "\n".join(out)
