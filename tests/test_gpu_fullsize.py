"""Configs 3 and 4 at their full sizes, in the launch configuration bench.py times: properties that hold at
any size on every layer, and the oracle on sampled layers (each of which it can compute in seconds).  The sample
follows the data: the layers where the GPU reports the most Sinkhorn iterations, a capped solve, the most
matching and auction rounds and the most moved tokens, plus three fixed ones."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from helpers import check_sinkhorn_problem, cpu, make_planner, oracle_schedule_layer, topology

pytestmark = pytest.mark.gpu


def _data_driven_sample(out, fixed):
    """Layers worth the oracle's time, chosen from the GPU's own outputs (each reason named for the failure text)."""
    it = cpu(out["sinkhorn_iters"]); info = cpu(out["info"]); rounds = cpu(out["rounds"])
    moved = cpu(out["X"].sum((1, 2)))
    picks = {"most Sinkhorn iterations": int(it.argmax()), "fewest Sinkhorn iterations": int(it.argmin()),
             "most auction rounds": int(rounds[:, 1].argmax()), "most matching rounds": int(rounds[:, 0].argmax()),
             "most moved tokens": int(moved.argmax())}
    capped = np.nonzero(info & 2)[0]
    if len(capped):
        picks["stopped at the iteration cap"] = int(capped[len(capped) // 2])
    for f in fixed:
        picks[f"fixed layer {f}"] = int(f)
    chosen = {}
    for why, l in picks.items():
        chosen.setdefault(l, why)
    return chosen


@pytest.mark.parametrize("name,fixed", [("cfg3", (0, 31, 57)), ("cfg4", (0, 23, 47))])
def test_full_size(name, fixed):
    cfg = W.get_config(name)
    e2r, C = topology(cfg)
    B = O.default_preference(C.numpy())
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg)
    out = pl.plan(topk)
    torch.cuda.synchronize()
    L, R, E, K, S, T, k = cfg.L, cfg.R, cfg.E, cfg.K, cfg.S, cfg.T, cfg.k
    # ---- every layer, on the GPU
    assert int(out["n"].sum()) == L * T * k and int(out["info"].bitwise_and(1).sum()) == 0
    assert torch.equal(out["n"].sum(1), out["expert_load"])
    ones = torch.ones_like(topk[0].reshape(-1))
    for l in range(L):
        el = torch.zeros(E, dtype=torch.int32, device="cuda").index_add_(0, topk[l].reshape(-1).long(), ones)
        assert torch.equal(el, out["expert_load"][l])
    ex = out["excess"].double(); sp = out["spare"].double()
    assert torch.equal(ex.sum(1), sp.sum(1))                                     # T*k divisible by R: balanced masses
    col_viol = (out["plan"].double().sum(1) - sp).abs().sum(1)
    assert bool((col_viol <= 1e-5 * ex.sum(1)).all()) and bool((out["plan"] >= 0).all())
    conv = (out["info"] & 2) == 0
    row_viol = (out["plan"].double().sum(2) - ex).abs().sum(1)
    assert bool((row_viol[conv] <= (1e-6 + 5e-7 + 1e-5) * ex.sum(1)[conv]).all())
    assert bool((out["X"].sum(1) == out["slot_tokens"].reshape(L, S)).all())     # every slot fully collected
    moved = out["new_idx"] != topk
    assert int(moved.sum()) == int(out["X"].sum())                               # token conservation
    assert bool((out["new_idx"][moved] >= E).all()) and bool((out["new_idx"][~moved] == topk[~moved]).all())
    again = pl.plan(topk)
    torch.cuda.synchronize()
    for key in ("plan", "X", "new_idx", "sinkhorn_iters"):
        assert torch.equal(again[key], out[key]), key                            # deterministic
    # ---- report and dispatch metadata at full size: properties on every layer
    rep = pl.report(out["expert_load"], out["rank_load"], out["slot_expert"], out["X"], 3.0)
    dsp = pl.dispatch(out["new_idx"])
    torch.cuda.synchronize()
    assert (cpu(rep["load_after"]).sum(1) == L * 0 + T * k).all() and (rep["rerouted"] == cpu(out["X"].sum((1, 2)))).all()
    assert torch.equal(dsp["send_counts"].sum(1), rep["load_after"])             # what a rank receives = its projected load
    assert torch.equal(dsp["target_counts"][:, :, E:], out["X"])                 # guest-slot columns = the auction's X
    seg = T // R * k
    e2r_d = e2r.cuda().long()
    for l in range(L):
        new = out["new_idx"][l].reshape(R, seg).long()
        dest = torch.where(new < E, e2r_d[new.clamp(max=E - 1)], (new - E) // K)
        key = dest * (E + S) + new
        perm = dsp["perm"][l].reshape(R, seg).long()
        buf = torch.empty_like(key).scatter_(1, perm, key)                       # the send buffer, by position
        assert bool((buf[:, 1:] >= buf[:, :-1]).all())                           # ordered by (destination, target)
        order = torch.empty_like(perm).scatter_(1, perm, torch.arange(seg, device="cuda").expand(R, seg))
        same = buf[:, 1:] == buf[:, :-1]
        assert bool((order[:, 1:][same] > order[:, :-1][same]).all())            # stable among equal keys
        assert bool((torch.sort(perm, dim=1).values == torch.arange(seg, device="cuda")).all())   # a permutation
    # ---- sampled layers against the oracle
    sample = _data_driven_sample(out, fixed)
    print(f"{name}: oracle on layers {sample}")
    assert 3 <= len(sample) <= 9
    for l in sample:
        tk = cpu(topk[l:l + 1])
        n, el, rl, bad = O.histogram(tk, R, E, e2r.numpy())
        assert (cpu(out["n"][l]) == n[0]).all() and (cpu(out["rank_load"][l]) == rl[0]).all()
        mean, exo, spo = O.excess_spare(rl)
        plan = cpu(out["plan"][l])
        check_sinkhorn_problem(exo[0].astype(np.float32), spo[0].astype(np.float32), C.numpy(), cfg.eps, plan,
                               int(out["sinkhorn_iters"][l]), float(out["row_err"][l]), cfg.max_iters, cfg.tol)
        m, a = oracle_schedule_layer(cfg, e2r.numpy(), B, n[0], el[0], rl[0], plan)
        assert (cpu(out["slot_expert"][l]).ravel() == m["slot_expert"]).all()
        assert (cpu(out["X"][l]) == a["X"]).all()
        assert cpu(out["rounds"][l]).tolist() == [m["inner_rounds"], a["rounds"]]
        want = O.assign(tk[0], R, E, K, m["slot_expert"], a["X"])
        assert (cpu(out["new_idx"][l]) == want).all()
        wd = O.dispatch(want, R, E, K, e2r.numpy())
        assert (cpu(dsp["perm"][l]) == wd["perm"]).all() and (cpu(dsp["send_counts"][l]) == wd["send_counts"]).all()
        wr = O.report(R, E, K, e2r.numpy(), C.numpy(), B, el[0], rl[0], m["slot_expert"], a["X"], 3.0)
        assert all(int(rep[key][l]) == wr[key] for key in O.REPORT_INTS)
        assert all(float(rep[key][l]) == wr[key] for key in O.REPORT_REALS)
    pl.close()
