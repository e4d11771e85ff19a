"""GPU parity of the dispatch report and of the two ablation switches against the oracle, on the
benchmark shapes and on the one-hot-rank imbalance workloads."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from helpers import check_sinkhorn_problem, cpu, make_planner, topology

pytestmark = pytest.mark.gpu

REPORT_CASES = {
    "cfg1": W.get_config("cfg1"),
    "cfg2": W.get_config("cfg2").replace(L=6),
    "cfg4_small": W.get_config("cfg4").replace(L=2, T=256 * 2304),
    "llep32": W.get_config("llep32"),
    "ladder16": W.get_config("ladder16"),
}


def _check_report(cfg, pl, out, lam):
    import paper_2608_03676_b200 as P
    e2r, C = topology(cfg)
    B = O.default_preference(C.numpy())
    rep = pl.report(out["expert_load"], out["rank_load"], out["slot_expert"], out["X"], lam)
    torch.cuda.synchronize()
    assert pl.last_launch_count() == 1
    o = {k: cpu(v) for k, v in out.items()}
    for l in range(cfg.L):
        want = O.report(cfg.R, cfg.E, cfg.K, e2r.numpy(), C.numpy(), B, o["expert_load"][l], o["rank_load"][l],
                        o["slot_expert"][l], o["X"][l], lam)
        for key in O.REPORT_INTS:
            assert int(rep[key][l]) == want[key], (l, key)
        for key in O.REPORT_REALS:
            assert float(rep[key][l]) == want[key], (l, key)         # single IEEE operations: same bits
        for key in ("spill", "load_after", "slot_moved", "slot_kind"):
            assert (cpu(rep[key])[l] == want[key]).all(), (l, key)
    text = P.format_layer(rep, 0, out["rank_load"], out["expert_load"], out["slot_expert"], e2r, cfg.K)
    assert "(1) load before" in text and "(4) imbalance" in text
    return rep


@pytest.mark.parametrize("name", list(REPORT_CASES))
def test_report_bit_exact(name):
    cfg = REPORT_CASES[name]
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg)
    out = pl.plan(topk)
    rep = _check_report(cfg, pl, out, 3.0)
    _check_report(cfg, pl, out, 2.5)
    # the plan reduces the imbalance and conserves the tokens
    assert (rep["rho_after"] <= rep["rho_before"]).all()
    assert (cpu(rep["load_after"]).sum(1) == rep["total_load"]).all()
    print(name, "rho", np.round(100 * rep["rho_before"], 2).tolist(), "->", np.round(100 * rep["rho_after"], 2).tolist())
    pl.close()


def test_report_optional_outputs_and_errors():
    import ctypes
    import paper_2608_03676_b200 as P
    cfg = W.get_config("cfg1")
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg)
    out = pl.plan(topk)
    rows = torch.zeros((cfg.L, 128), dtype=torch.uint8, device="cuda")
    ptr = lambda t: ctypes.c_void_p(t.data_ptr())
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = pl.lib.taot_report(pl.handle, ptr(out["expert_load"]), ptr(out["rank_load"]), ptr(out["slot_expert"]),
                            ptr(out["X"]), ctypes.c_double(3.0), ptr(rows), None, None, None, None, st)
    assert rc == 0
    torch.cuda.synchronize()
    full = pl.report(out["expert_load"], out["rank_load"], out["slot_expert"], out["X"], 3.0)
    rec = P.ReportRow.from_buffer_copy(rows.cpu().numpy().tobytes()[:128])
    assert rec.rerouted == int(full["rerouted"][0]) and rec.rho_after == float(full["rho_after"][0])
    assert ctypes.sizeof(P.ReportRow) == 128
    assert pl.lib.taot_report(pl.handle, None, ptr(out["rank_load"]), ptr(out["slot_expert"]), ptr(out["X"]),
                              ctypes.c_double(3.0), ptr(rows), None, None, None, None, st) == -1
    assert pl.lib.taot_report(pl.handle, ptr(out["expert_load"]), ptr(out["rank_load"]), ptr(out["slot_expert"]),
                              ptr(out["X"]), ctypes.c_double(float("nan")), ptr(rows), None, None, None, None, st) == -2
    assert pl.lib.taot_report(pl.handle, ptr(out["expert_load"]), ptr(out["rank_load"]), ptr(out["slot_expert"]),
                              ptr(out["X"]), ctypes.c_double(3.0), ctypes.c_void_p(rows.data_ptr() + 4), None, None,
                              None, None, st) == -5
    pl.close()


ABLATION_CASES = {
    "cfg2": W.get_config("cfg2").replace(L=6),
    "cfg3_small": W.get_config("cfg3").replace(L=2, T=64 * 2560),
    "ladder32": W.get_config("ladder32").replace(L=5),
}


@pytest.mark.parametrize("name", list(ABLATION_CASES))
@pytest.mark.parametrize("hint,topo", [(False, False), (False, True), (True, False)])
def test_ablation_switches_bit_exact(name, hint, topo):
    import paper_2608_03676_b200 as P
    cfg = ABLATION_CASES[name]
    e2r, C = topology(cfg)
    topk = W.routing_topk(cfg, device="cuda")
    flags = (0 if hint else P.ABLATE_HINT) | (0 if topo else P.ABLATE_TOPOLOGY)
    pl = make_planner(cfg, ablation=flags)
    out = {k: cpu(v) for k, v in pl.plan(topk).items()}
    assert pl.last_launch_count() == pl.plan_launches()
    assert pl.plan_launches() == (P.PLAN_LAUNCHES if hint else P.PLAN_LAUNCHES_NO_HINT)
    B = O.default_preference(C.numpy())
    B2 = B if topo else np.zeros_like(B)
    tk = cpu(topk)
    for l in range(cfg.L):
        if hint:
            check_sinkhorn_problem(out["excess"][l].astype(np.float32), out["spare"][l].astype(np.float32), C.numpy(),
                                   cfg.eps, out["plan"][l], out["sinkhorn_iters"][l], out["row_err"][l],
                                   cfg.max_iters, cfg.tol)
            hint_plan = out["plan"][l]
        else:
            assert (out["plan"][l] == 0).all() and out["sinkhorn_iters"][l] == 0 and out["row_err"][l] == 0
            hint_plan = np.zeros((cfg.R, cfg.R), np.float32)
        mean, ex, sp = O.excess_spare(out["rank_load"][l][None])
        spl = O.spill(out["expert_load"][l], e2r.numpy(), cfg.R, mean[0])
        m = O.match(cfg.R, cfg.E, cfg.K, e2r.numpy(), mean[0], ex[0], spl, sp[0], B2, hint_plan)
        a = O.auction(cfg.R, cfg.E, cfg.K, out["n"][l], m["slot_expert"], m["slot_tokens"], B)   # Phase 3 keeps B
        assert (out["slot_expert"][l].ravel() == m["slot_expert"]).all()
        assert (out["slot_tokens"][l].ravel() == m["slot_tokens"]).all()
        assert (out["X"][l] == a["X"]).all()
        assert out["rounds"][l].tolist() == [m["inner_rounds"], a["rounds"]]
        want = O.assign(tk[l], cfg.R, cfg.E, cfg.K, m["slot_expert"], a["X"])
        assert (out["new_idx"][l] == want).all()
    # the standalone matching call accepts a missing plan when the hint is switched off
    if not hint:
        dev = {k: torch.from_numpy(out[k]).cuda() for k in ("n", "expert_load", "rank_load")}
        m2 = pl.match(dev["n"], dev["expert_load"], dev["rank_load"], None)
        assert (cpu(m2["slot_expert"]) == out["slot_expert"]).all() and (cpu(m2["X"]) == out["X"]).all()
    pl.close()


def test_ablation_rejects_unknown_bits_and_full_method_needs_a_plan():
    import paper_2608_03676_b200 as P
    cfg = W.get_config("cfg1")
    with pytest.raises(P.TaotError):
        make_planner(cfg, ablation=4)
    pl = make_planner(cfg)
    out = pl.plan(W.routing_topk(cfg, device="cuda"))
    with pytest.raises(P.TaotError):
        pl.match(out["n"], out["expert_load"], out["rank_load"], None)
    pl.close()


def test_one_hot_rank_workloads_full_path_parity():
    """The imbalance-ladder workloads through the whole planner, all stages against the oracle."""
    for name in ("llep32", "ladder32"):
        cfg = W.get_config(name).replace(L=4)
        e2r, C = topology(cfg)
        topk = W.routing_topk(cfg, device="cuda")
        pl = make_planner(cfg)
        out = {k: cpu(v) for k, v in pl.plan(topk).items()}
        tk = cpu(topk)
        n, el, rl, bad = O.histogram(tk, cfg.R, cfg.E, e2r.numpy())
        assert (out["n"] == n).all() and (out["rank_load"] == rl).all() and (out["info"] & ~2 == 0).all()
        B = O.default_preference(C.numpy())
        for l in range(cfg.L):
            check_sinkhorn_problem(out["excess"][l].astype(np.float32), out["spare"][l].astype(np.float32), C.numpy(),
                                   cfg.eps, out["plan"][l], out["sinkhorn_iters"][l], out["row_err"][l],
                                   cfg.max_iters, cfg.tol)
            mean, ex, sp = O.excess_spare(rl[l][None])
            spl = O.spill(el[l], e2r.numpy(), cfg.R, mean[0])
            m = O.match(cfg.R, cfg.E, cfg.K, e2r.numpy(), mean[0], ex[0], spl, sp[0], B, out["plan"][l])
            a = O.auction(cfg.R, cfg.E, cfg.K, n[l], m["slot_expert"], m["slot_tokens"], B)
            assert (out["slot_expert"][l].ravel() == m["slot_expert"]).all() and (out["X"][l] == a["X"]).all()
            assert (out["new_idx"][l] == O.assign(tk[l], cfg.R, cfg.E, cfg.K, m["slot_expert"], a["X"])).all()
        pl.close()


def test_measured_alu_peaks_are_plausible():
    """The FMA and ex2 ceilings used as roofline denominators: within a factor of the figures that the SM
    count and clock imply (128 FMA lanes and 16 special-function lanes per SM per clock)."""
    import paper_2608_03676_b200 as P
    pk = P.measure_alu_peaks()
    props = torch.cuda.get_device_properties(0)
    clock_hz = 1.965e9
    fma_nominal = props.multi_processor_count * 128 * 2 * clock_hz / 1e12
    ex2_nominal = props.multi_processor_count * 16 * clock_hz / 1e12
    assert 0.5 * fma_nominal < pk["fma_tflops"] < 1.1 * fma_nominal, pk
    assert 0.5 * ex2_nominal < pk["ex2_tops"] < 1.1 * ex2_nominal, pk
    print(pk, fma_nominal, ex2_nominal)


def test_measured_latencies_are_plausible():
    """Dependent-operation latencies used for the chain floor of a Sinkhorn iteration: a fused multiply-add takes a
    few cycles, a shuffle-reduction level and a reciprocal-and-multiply a few tens; the same call twice agrees."""
    import paper_2608_03676_b200 as P
    a = P.measure_latencies()
    b = P.measure_latencies()
    assert 2.0 < a["fma"] < 12.0, a
    assert 10.0 < a["shuffle_level"] < 80.0, a
    assert 8.0 < a["rcp_mul"] < 80.0, a
    for key in a:
        assert abs(a[key] - b[key]) <= 0.15 * a[key] + 1.0, (a, b)


def test_measured_round_latencies_are_plausible():
    """Latencies of the operations an auction round chains: a shared-memory load and a barrier over eight warps take a
    few tens of cycles, an atomic with its result waited for somewhat more, and the arbitration triple (atomic,
    barrier, read-back) at least as long as a barrier plus a load less the overlap; the same call twice agrees."""
    import paper_2608_03676_b200 as P
    a = P.measure_round_latencies()
    b = P.measure_round_latencies()
    assert 10.0 < a["shared_load"] < 80.0, a
    assert 10.0 < a["shared_atomic"] < 300.0, a
    assert 10.0 < a["barrier"] < 300.0, a
    assert a["arbitration"] > max(a["barrier"], a["shared_load"]), a
    assert a["arbitration"] < a["shared_atomic"] + a["barrier"] + 2 * a["shared_load"] + 50.0, a
    for key in a:
        assert abs(a[key] - b[key]) <= 0.15 * a[key] + 2.0, (a, b)
