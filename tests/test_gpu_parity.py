"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Integer stages bit-exact; Sinkhorn within the stated tolerances."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from helpers import (check_sinkhorn_problem, cpu, make_planner, oracle_schedule_layer, topology)

pytestmark = pytest.mark.gpu

CASES = {
    # name: (config, overrides) -- sized so the oracle finishes in seconds, still several chunks + a ragged tail
    "cfg1": (W.get_config("cfg1"), {}),
    "cfg2": (W.get_config("cfg2"), {}),
    "cfg3_small": (W.get_config("cfg3").replace(L=3, T=64 * 2560), {}),      # SEG = 20480: 2 chunks, ragged
    "cfg4_small": (W.get_config("cfg4").replace(L=2, T=256 * 2304), {}),     # SEG = 18432: 2 chunks, ragged
}


def _routing(cfg):
    return W.routing_topk(cfg, device="cuda")


@pytest.fixture(scope="module", params=list(CASES))
def case(request):
    cfg, over = CASES[request.param]
    topk = _routing(cfg)
    pl = make_planner(cfg, **over)
    out = pl.plan(topk)
    torch.cuda.synchronize()
    yield cfg, topk, pl, {k: cpu(v) for k, v in out.items()}
    pl.close()


def test_histogram_bit_exact(case):
    cfg, topk, pl, out = case
    e2r, _ = topology(cfg)
    n, el, rl, bad = O.histogram(cpu(topk), cfg.R, cfg.E, e2r.numpy())
    assert (out["n"] == n).all() and (out["expert_load"] == el).all() and (out["rank_load"] == rl).all()
    assert (bad == 0).all() and ((out["info"] & 1) == 0).all()
    # the standalone entry point gives the same
    n2, el2, rl2, info2 = pl.histogram(topk)
    assert (cpu(n2) == n).all() and (cpu(el2) == el).all() and (cpu(rl2) == rl).all() and (cpu(info2) == 0).all()


def test_excess_spare_bit_exact(case):
    cfg, topk, pl, out = case
    mean, ex, sp = O.excess_spare(out["rank_load"])
    assert (out["excess"] == ex).all() and (out["spare"] == sp).all()
    ex2, sp2, s2, d2 = pl.excess_spare(torch.from_numpy(out["rank_load"]).cuda())
    assert (cpu(ex2) == ex).all() and (cpu(sp2) == sp).all()
    assert (cpu(s2) == ex.astype(np.float32)).all() and (cpu(d2) == sp.astype(np.float32)).all()


def test_sinkhorn_within_tolerance(case):
    cfg, topk, pl, out = case
    _, C = topology(cfg)
    worst = 0.0
    for l in range(cfg.L):
        s = out["excess"][l].astype(np.float32); d = out["spare"][l].astype(np.float32)
        r = check_sinkhorn_problem(s, d, C.numpy(), cfg.eps, out["plan"][l], out["sinkhorn_iters"][l],
                                   out["row_err"][l], cfg.max_iters, cfg.tol)
        worst = max(worst, r["max_rel"])
        capped = bool(out["info"][l] & 2)
        assert capped == (cfg.tol > 0 and out["sinkhorn_iters"][l] == cfg.max_iters and out["row_err"][l] > cfg.tol)
    print(f"{cfg.name}: worst plan rel err {worst:.2e}, iters {out['sinkhorn_iters'].tolist()}")


def test_schedule_bit_exact_given_the_gpu_plan(case):
    cfg, topk, pl, out = case
    e2r, C = topology(cfg)
    B = O.default_preference(C.numpy())
    for l in range(cfg.L):
        m, a = oracle_schedule_layer(cfg, e2r.numpy(), B, out["n"][l], out["expert_load"][l], out["rank_load"][l],
                                     out["plan"][l])
        assert (out["slot_expert"][l].ravel() == m["slot_expert"]).all()
        assert (out["slot_tokens"][l].ravel() == m["slot_tokens"]).all()
        assert (out["X"][l] == a["X"]).all()
        assert out["rounds"][l].tolist() == [m["inner_rounds"], a["rounds"]]
        assert a["residual"] == 0 and not (out["info"][l] & 8)
    print(f"{cfg.name}: rounds {out['rounds'].tolist()}")


def test_assign_bit_exact(case):
    cfg, topk, pl, out = case
    tk = cpu(topk)
    for l in range(cfg.L):
        want = O.assign(tk[l], cfg.R, cfg.E, cfg.K, out["slot_expert"][l].ravel(), out["X"][l])
        assert (out["new_idx"][l] == want).all()
    # standalone call, recounting the chunks itself, and reusing the histogram's counts
    se = torch.from_numpy(out["slot_expert"]).cuda(); X = torch.from_numpy(out["X"]).cuda()
    new, info = pl.assign(topk, se, X, reuse_counts=False)
    assert (cpu(new) == out["new_idx"]).all() and (cpu(info) == 0).all()
    pl.histogram(topk)
    new, info = pl.assign(topk, se, X, reuse_counts=True)
    assert (cpu(new) == out["new_idx"]).all()


def test_stage_calls_equal_the_chained_plan(case):
    cfg, topk, pl, out = case
    n, el, rl, _ = pl.histogram(topk)
    ex, sp, s, d = pl.excess_spare(rl)
    sk = pl.sinkhorn(s, d)
    assert (cpu(sk["plan"]) == out["plan"]).all() and (cpu(sk["iters"]) == out["sinkhorn_iters"]).all()
    m = pl.match(n, el, rl, sk["plan"])
    assert (cpu(m["slot_expert"]) == out["slot_expert"]).all() and (cpu(m["X"]) == out["X"]).all()
    assert pl.last_launch_count() >= 1


def test_plan_is_deterministic(case):
    cfg, topk, pl, out = case
    again = pl.plan(topk)
    torch.cuda.synchronize()
    for key, val in again.items():
        assert (cpu(val) == out[key]).all(), key
    import paper_2608_03676_b200 as P
    assert pl.last_launch_count() == pl.plan_launches() == P.PLAN_LAUNCHES


def test_plan_host_round_trip(case):
    cfg, topk, pl, out = case
    host_in = topk.cpu().pin_memory()
    host_out = pl.alloc_host_outputs(("n", "plan", "slot_expert", "slot_tokens", "X", "new_idx", "info", "rounds"))
    pl.plan_host(host_in, host_out)
    torch.cuda.synchronize()
    for key, val in host_out.items():
        assert (val.numpy() == out[key]).all(), key


def test_auction_dense_scan_with_an_untiered_preference_matrix():
    """A preference matrix with many distinct values takes the dense scan of Phase 3 instead of the
    tier bit sets; both must agree with the oracle bit for bit."""
    cfg = W.get_config("cfg2").replace(L=4)
    e2r, C = topology(cfg)
    g = torch.Generator().manual_seed(5)
    B = torch.rand((cfg.R, cfg.R), generator=g, dtype=torch.float32)
    B.fill_diagonal_(0.0)
    topk = _routing(cfg)
    pl = make_planner(cfg, B=B)
    out = {k: cpu(v) for k, v in pl.plan(topk).items()}
    for l in range(cfg.L):
        m, a = oracle_schedule_layer(cfg, e2r.numpy(), B.numpy(), out["n"][l], out["expert_load"][l],
                                     out["rank_load"][l], out["plan"][l])
        assert (out["slot_expert"][l].ravel() == m["slot_expert"]).all()
        assert (out["slot_tokens"][l].ravel() == m["slot_tokens"]).all()
        assert (out["X"][l] == a["X"]).all()
        assert out["rounds"][l].tolist() == [m["inner_rounds"], a["rounds"]]
    pl.close()


def test_auction_scores_that_round_together_and_a_round_cap():
    """A price step so small that different win counts give the same fp32 score (ties must then go to
    the lowest rank index, as in a dense scan), and a fixed number of auction rounds."""
    cfg = W.get_config("cfg2").replace(L=3)
    e2r, C = topology(cfg)
    B = O.default_preference(C.numpy())
    topk = _routing(cfg)
    for step, cap in ((1e-9, 0), (0.1, 5), (0.0, 0)):
        pl = make_planner(cfg, price_step=step, auction_max_rounds=cap)
        out = {k: cpu(v) for k, v in pl.plan(topk).items()}
        for l in range(cfg.L):
            m, a = oracle_schedule_layer(cfg, e2r.numpy(), B, out["n"][l], out["expert_load"][l],
                                         out["rank_load"][l], out["plan"][l], price_step=step,
                                         auction_max_rounds=cap)
            assert (out["X"][l] == a["X"]).all()
            assert out["rounds"][l, 1] == a["rounds"]
            assert bool(out["info"][l] & 8) == (a["residual"] > 0)
        pl.close()


@pytest.mark.parametrize("step", [0.0625, 0.25, 1.0 / 3.0, -0.05])
def test_auction_price_steps_with_ties_across_tiers(step):
    """Price steps that make scores of different tiers coincide exactly (1 - 15/16 = 1/16 is both the intra-node
    bonus after 15 wins and the far-tier bonus of the three-tier cost), a coarse and an inexact step, and a negative
    one (dense scan): the auction must follow the oracle bit for bit in every case."""
    for cfg in (W.get_config("cfg4").replace(L=2, T=256 * 2304), W.get_config("cfg2").replace(L=3)):
        e2r, C = topology(cfg)
        B = O.default_preference(C.numpy())
        topk = _routing(cfg)
        pl = make_planner(cfg, price_step=step)
        out = {k: cpu(v) for k, v in pl.plan(topk).items()}
        for l in range(cfg.L):
            m, a = oracle_schedule_layer(cfg, e2r.numpy(), B, out["n"][l], out["expert_load"][l],
                                         out["rank_load"][l], out["plan"][l], price_step=step)
            assert (out["X"][l] == a["X"]).all()
            assert out["rounds"][l, 1] == a["rounds"]
            assert bool(out["info"][l] & 8) == (a["residual"] > 0)
        pl.close()


def test_plan_is_capturable_in_a_cuda_graph():
    """taot_plan neither allocates nor synchronises, so a stream capture of it replays to the same bits
    (the paper stresses CUDA-graph compatibility of the planner, Appendix A.4)."""
    cfg = W.get_config("cfg2").replace(L=4)
    topk = _routing(cfg)
    pl = make_planner(cfg)
    out = pl.alloc_outputs()
    pl.plan(topk, out)
    torch.cuda.synchronize()
    want = {k: cpu(v).copy() for k, v in out.items()}
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        pl.plan(topk, out)                       # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        pl.plan(topk, out)
    for _ in range(3):
        for v in out.values():
            v.zero_()
        g.replay()
        torch.cuda.synchronize()
        for key, val in out.items():
            assert (cpu(val) == want[key]).all(), key
    # new routing written into the captured input buffer is planned by the next replay
    cfg2 = cfg.replace(seed=cfg.seed + 1)
    topk2 = _routing(cfg2)
    fresh = {k: cpu(v).copy() for k, v in pl.plan(topk2).items()}
    topk.copy_(topk2)
    g.replay()
    torch.cuda.synchronize()
    for key, val in out.items():
        assert (cpu(val) == fresh[key]).all(), key
    pl.close()


@pytest.mark.parametrize("base,over,L,G", [("cfg3", {}, 9, 4), ("cfg3", {}, 13, 6), ("cfg4", dict(T=256 * 2048), 12, 6)])
def test_layer_groups_on_internal_streams_change_no_bit_and_can_be_captured(monkeypatch, base, over, L, G):
    """A routing table large enough to be bandwidth-bound makes taot_plan split the layers into groups on streams of
    its own (fork / join by events).  The split must change no output, it must be capturable in a CUDA graph, and the
    group timeline must show every group passing through the five stages in order.  At 256 ranks the one-byte copies of
    the groups' tables are made on one more stream after the histograms, and the reassignments wait for them."""
    cfg = W.get_config(base).replace(L=L, **over)        # L x 64 x 4 chunks: 9 layers make four groups, 13 make six
    topk = _routing(cfg)
    monkeypatch.setenv("TAOT_PLAN_GROUPS", "1")
    single = make_planner(cfg)
    monkeypatch.delenv("TAOT_PLAN_GROUPS")
    pl = make_planner(cfg)
    want = {k: cpu(v).copy() for k, v in single.plan(topk).items()}
    out = pl.alloc_outputs()
    pl.plan(topk, out)
    torch.cuda.synchronize()
    n1 = single.last_launch_count()
    # G groups, the same kernels each; at 256 ranks the one-byte copy of each group's table is a launch of its own
    assert pl.last_launch_count() in (G * n1, G * (n1 + 1))
    for key, val in out.items():
        assert (cpu(val) == want[key]).all(), key
    pl.set_profiling(3)
    pl.plan(topk, out)
    trace = pl.group_trace()
    pl.set_profiling(0)
    assert len(trace) == G and single.group_trace() == []
    for row in trace:
        assert all(b >= a for a, b in zip(row, row[1:]))                     # stages in order
    assert all(trace[g + 1][1] >= trace[g][1] for g in range(G - 1))         # the histograms run one after the other
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        pl.plan(topk, out)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        pl.plan(topk, out)
    for _ in range(2):
        for v in out.values():
            v.zero_()
        g.replay()
        torch.cuda.synchronize()
        for key, val in out.items():
            assert (cpu(val) == want[key]).all(), key
    pl.close(); single.close()


def test_pipelined_host_planner_equals_the_single_call():
    import paper_2608_03676_b200 as P
    cfg = W.get_config("cfg2").replace(L=7)            # 7 layers over 3 groups: uneven split
    e2r, C = topology(cfg)
    topk = _routing(cfg)
    pl = make_planner(cfg)
    want = {k: cpu(v) for k, v in pl.plan(topk).items()}
    hp = P.PipelinedHostPlanner(L=cfg.L, groups=3, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r, C=C,
                                eps=cfg.eps, max_iters=cfg.max_iters, tol=cfg.tol)
    assert [hi - lo for lo, hi in hp.bounds] == [3, 2, 2]
    names = ("n", "plan", "sinkhorn_iters", "slot_expert", "slot_tokens", "X", "new_idx", "info", "rounds")
    host_out = hp.alloc_host_outputs(names)
    host_in = topk.cpu().pin_memory()
    for _ in range(2):
        for v in host_out.values():
            v.zero_()
        hp.plan_host(host_in, host_out)
        torch.cuda.synchronize()
        for key in names:
            assert (host_out[key].numpy() == want[key]).all(), key
    assert hp.launch_count() == hp.plan_launches() == 3 * P.PLAN_LAUNCHES
    hp.close(); pl.close()


@pytest.mark.parametrize("groups", [1, 2])
def test_streaming_host_planner_keeps_steps_apart(groups):
    """Two host calls in flight on alternating inputs: every step's outputs are those of a lone call on its input.
    With one group of layers per call the outputs are packed (one block and one copy for all but the routing
    table); with two, every output has its own buffer and copy."""
    import paper_2608_03676_b200 as P
    cfg = W.get_config("cfg2").replace(L=5)
    e2r, C = topology(cfg)
    pl = make_planner(cfg)
    inputs = [_routing(cfg.replace(seed=cfg.seed + i)) for i in range(3)]
    names = ("n", "plan", "sinkhorn_iters", "slot_expert", "slot_tokens", "X", "new_idx", "info", "rounds")
    want = [{k: cpu(v).copy() for k, v in pl.plan(t).items()} for t in inputs]
    assert (want[0]["new_idx"] != want[1]["new_idx"]).any()
    sp = P.StreamingHostPlanner(L=cfg.L, depth=2, groups=groups, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r,
                                C=C, eps=cfg.eps, max_iters=cfg.max_iters, tol=cfg.tol)
    outs = sp.alloc_host_outputs(names)
    assert ("_block" in outs[0]) == (groups == 1)
    host_in = [t.cpu().pin_memory() for t in inputs]
    tickets = []
    for step in range(7):
        which = step % 3
        if step >= 2:                                   # read the step that used this lane before submitting into it
            got = sp.result(tickets[step - 2][0])
            ref = want[tickets[step - 2][1]]
            for key in names:
                assert (got[key].numpy() == ref[key]).all(), (step, key)
        tickets.append((sp.submit(host_in[which], outs[step % 2]), which))
    for t, which in tickets[-2:]:
        got = sp.result(t)
        for key in names:
            assert (got[key].numpy() == want[which][key]).all(), (t, key)
    with pytest.raises(P.TaotError):
        sp.result(0)
    sp.close(); pl.close()
