"""Edge and degenerate cases of the CUDA path against the oracle: bad indices, balanced layers,
supply exceeding demand, unaligned / ragged routing tables, extreme cost/eps (hand-back and
log-domain paths of the Sinkhorn kernels), overlapping supply/demand supports, odd expert maps."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from helpers import check_sinkhorn_problem, cpu, make_planner, oracle_schedule_layer, topology

pytestmark = pytest.mark.gpu


def _full_check(cfg, topk, pl, B=None, e2r=None, C=None, expect_bad=False):
    """Plan on the GPU and compare every stage with the oracle (schedule fed the GPU plan)."""
    e2r_t, C_t = topology(cfg)
    e2r = e2r_t.numpy() if e2r is None else e2r
    C = C_t.numpy() if C is None else C
    Bm = O.default_preference(C) if B is None else B
    dev = pl.plan(topk)
    out = {k: cpu(v) for k, v in dev.items()}
    tk = cpu(topk)
    n, el, rl, bad = O.histogram(tk, cfg.R, cfg.E, e2r)
    assert (out["n"] == n).all() and (out["expert_load"] == el).all() and (out["rank_load"] == rl).all()
    assert ((out["info"] & 1) != 0).tolist() == (bad > 0).tolist()
    assert bool((bad > 0).any()) == expect_bad
    mean, ex, sp = O.excess_spare(rl)
    assert (out["excess"] == ex).all() and (out["spare"] == sp).all()
    for l in range(cfg.L):
        s = ex[l].astype(np.float32); d = sp[l].astype(np.float32)
        check_sinkhorn_problem(s, d, C, pl.params.eps, out["plan"][l], out["sinkhorn_iters"][l], out["row_err"][l],
                               pl.params.max_iters, pl.params.tol, pl.params.check_every)
        assert bool(out["info"][l] & 16) == (s.sum() > d.sum())
        m, a = oracle_schedule_layer(cfg, e2r, Bm, n[l], el[l], rl[l], out["plan"][l])
        assert (out["slot_expert"][l].ravel() == m["slot_expert"]).all()
        assert (out["slot_tokens"][l].ravel() == m["slot_tokens"]).all()
        assert (out["X"][l] == a["X"]).all()
        want = O.assign(tk[l], cfg.R, cfg.E, cfg.K, m["slot_expert"], a["X"])
        assert (out["new_idx"][l] == want).all()
    # the diagnostics and the dispatch metadata of the same plan
    rep = pl.report(dev["expert_load"], dev["rank_load"], dev["slot_expert"], dev["X"], 3.0)
    dsp = pl.dispatch(dev["new_idx"])
    torch.cuda.synchronize()
    for l in range(cfg.L):
        wr = O.report(cfg.R, cfg.E, cfg.K, e2r, C, Bm, el[l], rl[l], out["slot_expert"][l], out["X"][l], 3.0)
        for key in O.REPORT_INTS:
            assert int(rep[key][l]) == wr[key], (l, key)
        for key in O.REPORT_REALS:
            assert float(rep[key][l]) == wr[key], (l, key)
        for key in ("spill", "load_after", "slot_moved", "slot_kind"):
            assert (cpu(rep[key])[l] == wr[key]).all(), (l, key)
        wd = O.dispatch(out["new_idx"][l], cfg.R, cfg.E, cfg.K, e2r)
        assert (cpu(dsp["perm"])[l] == wd["perm"]).all()
        assert (cpu(dsp["send_counts"])[l] == wd["send_counts"]).all()
        assert (cpu(dsp["target_counts"])[l] == wd["target_counts"]).all()
        assert bool(cpu(dsp["info"])[l] & 1) == (wd["bad"] > 0)
    return out


def test_out_of_range_indices_are_skipped_flagged_and_copied_through():
    cfg = W.get_config("cfg2").replace(L=3)
    topk = W.routing_topk(cfg, device="cuda")
    topk[1, 5, 2] = -1
    topk[1, 9000, 0] = cfg.E
    topk[2, 16383, 7] = 2 ** 30
    pl = make_planner(cfg)
    out = _full_check(cfg, topk, pl, expect_bad=True)
    assert out["info"][0] & 1 == 0 and out["info"][1] & 1 and out["info"][2] & 1
    assert out["new_idx"][1, 5, 2] == -1 and out["new_idx"][1, 9000, 0] == cfg.E and out["new_idx"][2, 16383, 7] == 2 ** 30
    pl.close()


def test_perfectly_balanced_layer_moves_nothing():
    cfg = W.get_config("cfg1").replace(L=2)
    topk = W.routing_topk(cfg, device="cuda")
    # layer 1: every token t picks experts (t mod E) and (t+1 mod E): all ranks carry the same load
    t = torch.arange(cfg.T, device="cuda")
    topk[1, :, 0] = (t % cfg.E).int()
    topk[1, :, 1] = ((t + 1) % cfg.E).int()
    pl = make_planner(cfg)
    out = _full_check(cfg, topk, pl)
    assert (out["excess"][1] == 0).all() and (out["plan"][1] == 0).all() and out["sinkhorn_iters"][1] == 0
    assert (out["slot_expert"][1] == -1).all() and (out["X"][1] == 0).all()
    assert (out["new_idx"][1] == cpu(topk)[1]).all()
    pl.close()


def test_total_load_not_divisible_by_ranks_scales_the_supply():
    # T*k = 3*1000*3 = 9000 entries over R = 7 ranks?  T must be a multiple of R: T = 7*143, k = 3 -> 3003 entries,
    # 3003 mod 7 = 0; use E = 7*3 experts but route one extra-heavy pattern so that sum(l) mod R != 0 is impossible
    # with every entry counted.  Bad indices are skipped, which makes the counted total non-divisible.
    cfg = W.get_config("cfg1").replace(L=2, R=7, E=21, K=2, k=3, T=7 * 143, gpus_per_node=4)
    topk = W.routing_topk(cfg, device="cuda")
    topk[0, 0, 0] = -5                      # one entry dropped: total = 3002, 3002 mod 7 = 6 -> sum(excess) > sum(spare)
    pl = make_planner(cfg, max_iters=300, tol=0.0)
    out = _full_check(cfg, topk, pl, expect_bad=True)
    assert out["info"][0] & 16 and out["excess"][0].sum() - out["spare"][0].sum() == 6
    pl.close()


@pytest.mark.parametrize("k,tpr,R,E", [(3, 1001, 4, 12), (5, 3333, 8, 16), (1, 40000, 2, 6), (8, 2049, 4, 8), (2, 70001, 2, 6),
                                       (4, 35000, 2, 6)])
def test_unaligned_and_ragged_segments(k, tpr, R, E):
    # SEG = tpr*k: not a multiple of 4 (scalar load path) and/or several chunks with a short last one (the last two
    # cases: nine chunks per segment, so a chunk's starting ordinals are sums over up to eight earlier chunks)
    cfg = W.get_config("cfg1").replace(L=2, R=R, E=E, K=2, k=k, T=R * tpr, gpus_per_node=2, zipf=(1.3, 1.3))
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg, max_iters=200, tol=1e-6)
    _full_check(cfg, topk, pl)
    # a routing table that does not start on a 16-byte boundary
    buf = torch.empty(topk.numel() + 1, dtype=torch.int32, device="cuda")
    shifted = buf[1:].view_as(topk)
    shifted.copy_(topk)
    n, el, rl, info = pl.histogram(shifted)
    n0, el0, rl0, _ = pl.histogram(topk)
    assert torch.equal(n, n0) and torch.equal(rl, rl0)
    out = pl.plan(topk)
    new, _ = pl.assign(shifted, out["slot_expert"], out["X"], reuse_counts=False)
    assert torch.equal(new, out["new_idx"])
    pl.close()


def test_uneven_expert_map_and_three_slots():
    cfg = W.get_config("cfg2").replace(L=3, K=3)
    e2r = torch.tensor([0] * 10 + [1] * 2 + [2] * 1 + [3] * 7 + list(range(4, 16)) * 3 + [15] * 8, dtype=torch.int32)
    assert e2r.numel() == cfg.E
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers)
    import paper_2608_03676_b200 as P
    pl = P.Planner(L=cfg.L, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r, C=C, eps=cfg.eps, max_iters=500,
                   tol=1e-6)
    topk = W.routing_topk(cfg, device="cuda")
    _full_check(cfg, topk, pl, e2r=e2r.numpy())
    pl.close()


@pytest.mark.parametrize("eps,iters,check_every", [(0.004, 150, 1), (0.02, 1, 1), (0.2, 400, 7)])
def test_extreme_cost_over_eps_single_iteration_and_sparse_checks(eps, iters, check_every):
    # eps = 0.004 gives C/eps up to 2500: far beyond fp32's exponent range
    cfg = W.get_config("cfg2").replace(L=6)
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg, eps=eps, max_iters=iters, tol=1e-6 if check_every > 1 else 0.0, check_every=check_every)
    _full_check(cfg, topk, pl)
    pl.close()


def test_overlapping_supports_and_many_supply_ranks_take_the_shared_memory_kernel():
    # taot_sinkhorn with arbitrary s, d: ranks with both supply and demand, more supply ranks than the register
    # tile holds (R = 64: 32 rows), zero rows, and a problem with no demand at all
    cfg = W.get_config("cfg3").replace(L=4, T=64 * 64)
    pl = make_planner(cfg, max_iters=120, tol=0.0)
    _, C = topology(cfg)
    g = torch.Generator().manual_seed(3)
    s = torch.rand((4, 64), generator=g) * 100
    d = torch.rand((4, 64), generator=g) * 100
    s[0, 40:] = 0; d[0, :24] = 0                       # 40 supply ranks (> 32), overlapping with demand on 24..39
    s[1, ::2] = 0                                      # overlapping supports everywhere else
    s[2] = 0; s[2, 5] = 7; d[2] = 0; d[2, 9] = 7       # 1 x 1 problem
    d[3] = 0                                           # nothing can move
    out = pl.sinkhorn(s.cuda(), d.cuda())
    torch.cuda.synchronize()
    for b in range(4):
        check_sinkhorn_problem(s[b].numpy(), d[b].numpy(), C.numpy(), cfg.eps, cpu(out["plan"])[b],
                               cpu(out["iters"])[b], cpu(out["row_err"])[b], 120, 0.0)
    assert cpu(out["iters"]).tolist() == [120, 120, 120, 0]
    pl.close()


def test_handle_validation_and_null_arguments_return_status_codes():
    import ctypes
    import paper_2608_03676_b200 as P
    cfg = W.get_config("cfg1")
    pl = make_planner(cfg)
    lib = P.load_library()
    topk = W.routing_topk(cfg, device="cuda")
    out = pl.alloc_outputs()
    assert lib.taot_histogram(pl.handle, None, None, None, None, None, None, None) == -1
    o = pl._outputs_struct(out)
    assert lib.taot_plan(pl.handle, ctypes.c_void_p(topk.data_ptr()), ctypes.byref(o), ctypes.c_void_p(pl.ws.data_ptr() + 4), None) == -5
    o.new_idx = topk.data_ptr()                         # in-place rewrite is refused
    assert lib.taot_plan(pl.handle, ctypes.c_void_p(topk.data_ptr()), ctypes.byref(o), ctypes.c_void_p(pl.ws.data_ptr()), None) == -2
    with pytest.raises(P.TaotError):
        pl.histogram(topk.cpu())                        # host tensor where device memory is required
    pl.close()


def test_many_quota_boundaries_inside_one_chunk():
    """A hand-made schedule in which ten guest slots hold the same expert and every source rank feeds each of
    them a few tokens: ten quota intervals end inside the single chunk of a segment, more than the four splits the
    rewrite applies from registers, so it walks the list of split records.  Checked through taot_assign alone."""
    cfg = W.get_config("cfg1").replace(L=2, R=8, E=8, K=4, k=2, T=8 * 4096)
    e2r, _ = topology(cfg)
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg)
    n, el, rl, _ = pl.histogram(topk)
    n_h = cpu(n)
    S = cfg.S
    slot_expert = np.full((cfg.L, S), -1, np.int32)
    X = np.zeros((cfg.L, cfg.R, S), np.int32)
    for l in range(cfg.L):
        e0 = int(np.argmax(n_h[l].sum(0)))                               # the busiest expert of the layer
        slots = [s for s in range(S) if s // cfg.K != e2r[e0]][:10]
        for q, s in enumerate(slots):
            slot_expert[l, s] = e0
            for r in range(cfg.R):
                X[l, r, s] = min(3 + (q + r) % 5, max(0, int(n_h[l, r, e0]) // 12))
        other = int(np.argsort(n_h[l].sum(0))[-2])                       # and one slot for the runner-up
        s2 = [s for s in range(S) if slot_expert[l, s] < 0 and s // cfg.K != e2r[other]][0]
        slot_expert[l, s2] = other
        X[l, :, s2] = np.minimum(n_h[l, :, other] // 3, 50)
    se_d = torch.from_numpy(slot_expert.reshape(cfg.L, cfg.R, cfg.K)).cuda()
    X_d = torch.from_numpy(X).cuda()
    for reuse in (True, False):
        if reuse:
            pl.histogram(topk)
        new, info = pl.assign(topk, se_d, X_d, reuse_counts=reuse)
        torch.cuda.synchronize()
        assert (cpu(info) == 0).all()
        for l in range(cfg.L):
            want = O.assign(cpu(topk)[l], cfg.R, cfg.E, cfg.K, slot_expert[l], X[l])
            assert (cpu(new)[l] == want).all()
            assert int((want >= cfg.E).sum()) == int(X[l].sum())
    pl.close()


def test_largest_supported_dimensions():
    """E = 1024 experts, K = 8 slots per rank, top-64 routing (the documented maxima) on 64 ranks: every stage,
    the report and the dispatch metadata against the oracle."""
    cfg = W.get_config("cfg1").replace(L=1, R=64, E=1024, K=8, k=64, T=64 * 96, gpus_per_node=8,
                                       tiers=(0.0, 1.0, 4.0), zipf=(1.1, 1.1))
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg, max_iters=300, tol=1e-6)
    out = _full_check(cfg, topk, pl)
    assert out["X"].sum() > 0
    pl.close()


def test_most_slots_256_ranks_by_8_slots():
    """S = 2048 guest slots (256 ranks x 8): more slots than the one-thread-per-slot auction holds, so Phase 3 takes
    the dense scan; the whole path, the report and the dispatch metadata against the oracle."""
    cfg = W.get_config("cfg4").replace(L=1, E=512, K=8, k=8, T=256 * 64, e2r_mode="contiguous", zipf=(1.3, 1.3))
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg, max_iters=200, tol=1e-6)
    out = _full_check(cfg, topk, pl)
    assert out["X"].sum() > 0
    pl.close()


def test_smallest_table_and_everything_on_one_expert():
    """One token per rank with top-1 routing (the smallest table the API accepts), and a layer in which every
    entry names the same expert (one rank holds the whole load, its other experts none)."""
    cfg = W.get_config("cfg1").replace(L=2, R=8, E=32, K=2, k=1, T=8)
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg, max_iters=100, tol=0.0)
    _full_check(cfg, topk, pl)
    pl.close()
    cfg = W.get_config("cfg1").replace(L=2, k=2, T=8 * 640)
    topk = W.routing_topk(cfg, device="cuda")
    topk[0, :, 0] = 5                          # layer 0: first choice always expert 5 ...
    topk[0, :, 1] = 5                          # ... and the second too (duplicates inside a token are legal input)
    pl = make_planner(cfg, max_iters=200, tol=1e-6)
    out = _full_check(cfg, topk, pl)
    assert out["rank_load"][0].max() == cfg.T * cfg.k and (out["slot_expert"][0] >= 0).sum() > 0
    pl.close()


@pytest.mark.parametrize("R,B", [(16, 6), (64, 5), (256, 4)])
def test_non_finite_supply_or_demand_is_flagged_on_its_problem_only(R, B):
    """taot_sinkhorn takes the caller's s and d: a NaN or an infinity in one entry of one problem must give that
    problem TAOT_INFO_NONFINITE, a zero plan and 0 iterations, leave its neighbours within tolerance, and trap
    nothing (the injection is on the host; the kernels only ever see bounded loops and data-independent indices)."""
    import paper_2608_03676_b200 as P
    from workloads.configs import SWEEP_TIERS
    C = W.cost_matrix(R, 8, SWEEP_TIERS, 4)
    eps = 0.1 * max(SWEEP_TIERS)
    pl = P.Planner(L=B, R=R, E=R, K=1, k=1, T=R, e2r=torch.arange(R, dtype=torch.int32), C=C, eps=eps,
                   max_iters=60, tol=0.0)
    loads = W.sweep_rank_loads(B, R, seed=123, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    s = s.clone(); d = d.clone()
    hot1 = int(torch.nonzero(s[1] > 0)[0]); cold2 = int(torch.nonzero(d[2] > 0)[-1])
    s[1, hot1] = float("nan")                        # problem 1: NaN supply
    d[2, cold2] = float("inf")                       # problem 2: infinite demand
    s[3, int(torch.nonzero(s[3] > 0)[-1])] = float("inf")   # problem 3: infinite supply
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    for b in (1, 2, 3):
        assert info[b] & P.INFO_NONFINITE and iters[b] == 0 and (plan[b] == 0).all(), b
    for b in [0] + list(range(4, B)):
        assert info[b] == 0 and iters[b] == 60
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), eps, plan[b], iters[b], err[b], 60, 0.0)
    # the context is alive and the handle still usable
    again = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    assert torch.equal(again["plan"], out["plan"])
    pl.close()


def test_supports_beyond_the_on_chip_capacity_at_256_ranks_are_flagged_not_solved():
    """At 256 ranks a problem whose |supply ranks| x |demand ranks| exceeds R*R/4 (possible only with overlapping
    supports, which the planner's own excess / spare never produce) gets TAOT_INFO_SINKHORN_SIZE and a zero plan;
    a problem at the limit and an ordinary one in the same batch are solved."""
    import paper_2608_03676_b200 as P
    R = 256
    C = W.cost_matrix(R, 8, (0.0, 1.0, 6.0, 16.0), 4)
    i = torch.arange(R)
    C = C + 0.25 * (((i[:, None] * 5 + i[None, :] * 3) % 11 == 0) & (i[:, None] != i[None, :])).float()   # general cost
    pl = P.Planner(L=3, R=R, E=R, K=1, k=1, T=R, e2r=torch.arange(R, dtype=torch.int32), C=C, eps=1.6,
                   max_iters=30, tol=0.0)
    g = torch.Generator().manual_seed(11)
    s = torch.zeros((3, R)); d = torch.zeros((3, R))
    s[0, :200] = torch.rand(200, generator=g) * 50 + 1; d[0, 56:] = torch.rand(200, generator=g) * 50 + 1   # 200 x 200 > 16384
    s[1, :128] = torch.rand(128, generator=g) * 50 + 1; d[1, 128:] = torch.rand(128, generator=g) * 50 + 1  # 128 x 128: the limit
    s[2, :20] = torch.rand(20, generator=g) * 50 + 1; d[2, 100:160] = torch.rand(60, generator=g) * 50 + 1
    out = pl.sinkhorn(s.cuda(), d.cuda())
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    assert info[0] & P.INFO_SINKHORN_SIZE and (plan[0] == 0).all()
    for b in (1, 2):
        assert (info[b] & P.INFO_SINKHORN_SIZE) == 0 and iters[b] == 30
        check_sinkhorn_problem(s[b].numpy(), d[b].numpy(), C.numpy(), 1.6, plan[b], iters[b], err[b], 30, 0.0)
    pl.close()


def test_negative_preference_entries_order_scores_as_floats_do():
    """A preference matrix with negative entries makes some Phase-2 scores negative; the integer key the kernel
    takes its arg-max over must still order them as the floating-point comparison of the oracle does."""
    cfg = W.get_config("cfg2").replace(L=4)
    e2r, C = topology(cfg)
    B = O.default_preference(C.numpy()).copy()
    g = np.random.default_rng(5)
    B[g.random(B.shape) < 0.3] *= -400.0             # alpha * B then outweighs any gain: negative scores compete
    np.fill_diagonal(B, 0.0)
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg, B=torch.from_numpy(B))
    _full_check(cfg, topk, pl, B=B)
    pl.close()
