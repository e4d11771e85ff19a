"""Config 5 (Sinkhorn-only scaling sweep): sampled cells against the oracle.  Rank loads come from
the sweep generator, supply/demand from `taot_excess_spare`, 500 fixed iterations, 3-tier cost."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from workloads.configs import SWEEP_ITERS, SWEEP_TIERS
from helpers import check_sinkhorn_problem, cpu

pytestmark = pytest.mark.gpu


def _planner(B, R, eps_frac, iters=SWEEP_ITERS, tol=0.0, general=False):
    """general: a few entries of the tiered cost are raised, so that it no longer depends on the tier alone and the
    solve takes the kernels that hold the kernel matrix itself (register tiles, clusters, workspace) instead of the
    tier-by-tier sums."""
    import paper_2608_03676_b200 as P
    C = W.cost_matrix(R, 8, SWEEP_TIERS, 4)
    if general:
        i = torch.arange(R)
        bump = ((i[:, None] * 5 + i[None, :] * 3) % 11 == 0) & (i[:, None] != i[None, :])
        C = C + 0.25 * bump.to(C.dtype)
    e2r = torch.arange(R, dtype=torch.int32)
    pl = P.Planner(L=B, R=R, E=R, K=1, k=1, T=R, e2r=e2r, C=C, eps=eps_frac * max(SWEEP_TIERS),
                   max_iters=iters, tol=tol)
    return pl, C


@pytest.mark.parametrize("R,B,check,general", [
    (8, 64, 64, False), (16, 64, 64, False), (64, 64, 16, False), (256, 64, 4, False), (1024, 3, 1, False),
    # batches of at least 4 x 148 problems take the batch builds of the kernels
    (16, 1024, 8, False), (64, 1024, 6, False), (256, 640, 3, False),
    # beyond 256 ranks with the tiered cost: tier-by-tier sums, eight warps per problem, 2 and 4 ranks per lane
    (512, 8, 2, False), (1024, 8, 1, False),
    # a cost that is not tiered: 16-warp register tile, 4-warp batch tile, clusters
    (256, 64, 3, True), (256, 640, 2, True), (1024, 3, 1, True)])
@pytest.mark.parametrize("eps_frac", [0.1, 0.01])
def test_sweep_cell(R, B, check, eps_frac, general):
    pl, C = _planner(B, R, eps_frac, general=general)
    loads = W.sweep_rank_loads(B, R, seed=1000 + R, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    mean, ex_ref, sp_ref = O.excess_spare(cpu(loads))
    assert (cpu(ex) == ex_ref).all() and (cpu(sp) == sp_ref).all()
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    assert (iters == SWEEP_ITERS).all() and (info == 0).all()
    worst = 0.0
    for b in range(check):
        r = check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), eps_frac * max(SWEEP_TIERS), plan[b], iters[b],
                                   err[b], SWEEP_ITERS, 0.0)
        worst = max(worst, r["max_rel"])
    # properties that hold for every problem of the cell, checked on the GPU
    tot = s.double().sum(1)
    col_viol = (out["plan"].double().sum(1) - d.double()).abs().sum(1)
    assert bool((col_viol <= 1e-5 * tot).all())
    assert bool((out["plan"] >= 0).all())
    print(f"R={R} eps={eps_frac}: worst rel err {worst:.2e} over {check} problems")
    pl.close()


@pytest.mark.parametrize("general", [True, False])
def test_large_batch_with_mixed_problem_sizes_walks_the_kernel_chain(general):
    """A batch that takes the 4-warp batch kernel, in which some problems have more supply ranks than that kernel
    holds (they must come back marked and be solved by the 16-warp kernel), in tolerance mode.  With the tiered
    cost the same batch goes through the tier-by-tier kernel, which has no such limit."""
    R, B = 256, 640
    pl, C = _planner(B, R, 0.1, iters=300, tol=1e-6, general=general)
    loads = W.sweep_rank_loads(B, R, seed=77, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(9)
    wide = torch.randint(1000, 60000, (B // 2, R), generator=g, device="cuda", dtype=torch.int32)
    loads[1::2] = wide                                   # every other problem: about half of the ranks above the mean
    ex, sp, s, d = pl.excess_spare(loads)
    hn = (ex > 0).sum(1)
    assert int(hn[0::2].max()) <= 32 < int(hn[1::2].min())      # some of the wide ones exceed 128 too: third kernel
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    assert (iters >= 1).all() and (iters <= 300).all() and ((info & ~(2 | 16)) == 0).all()   # 16: supply scaled (the integer mean leaves a remainder)
    for b in (0, 1, 2, 3, 638, 639):
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(SWEEP_TIERS), plan[b], iters[b], err[b],
                               300, 1e-6)
    tot = s.double().sum(1)
    col_viol = (out["plan"].double().sum(1) - d.double()).abs().sum(1)
    assert bool((col_viol <= 1e-5 * tot).all()) and bool((out["plan"] >= 0).all())
    pl.close()


@pytest.mark.parametrize("R", [512, 1024])
def test_cluster_kernel_and_its_fall_through_beyond_256_ranks(R):
    """About half of the ranks with supply: at 512 ranks the four-CTA clusters hold the problem, at 1024 ranks a
    slice of 128 rows x 512 columns does not fit and the problem falls through to the kernel with the matrix in
    workspace; one narrow problem beside it stays on the clusters.  Both against the oracle."""
    B = 3
    pl, C = _planner(B, R, 0.1, iters=40, tol=0.0, general=True)
    loads = W.sweep_rank_loads(B, R, seed=31, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(4)
    loads[1] = torch.randint(1000, 60000, (R,), generator=g, device="cuda", dtype=torch.int32)
    ex, sp, s, d = pl.excess_spare(loads)
    hn = (ex > 0).sum(1).tolist()
    assert hn[1] > R // 3 and hn[0] < R // 8
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    assert (iters == 40).all() and ((info & ~16) == 0).all()
    for b in range(B):
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(SWEEP_TIERS), plan[b], iters[b], err[b], 40, 0.0)
    pl.close()


def test_batches_larger_than_the_handle_and_unsupported_calls_beyond_256_ranks():
    import paper_2608_03676_b200 as P
    R = 512
    pl, C = _planner(2, R, 0.1, iters=20)
    loads = W.sweep_rank_loads(5, R, seed=7, device="cuda")        # 5 problems through a handle built for 2
    ex, sp, s, d = pl.excess_spare(loads)
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    for b in (0, 2, 4):
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(SWEEP_TIERS), cpu(out["plan"])[b],
                               cpu(out["iters"])[b], cpu(out["row_err"])[b], 20, 0.0)
    topk = torch.zeros((2, R, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(P.TaotError):
        pl.histogram(topk)
    pl.close()


def test_tiered_kernel_hands_back_a_rank_with_both_supply_and_demand():
    """The tier-by-tier sums leave out the diagonal, which is right only while no rank has both supply and demand;
    a problem that has such a rank must come back from that kernel and be solved by the general one."""
    R, B = 256, 4
    pl, C = _planner(B, R, 0.1, iters=60)
    loads = W.sweep_rank_loads(B, R, seed=5, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    s = s.clone(); d = d.clone()
    j = int(torch.nonzero(d[1] > 0)[0])
    s[1, j] = 7.0                                        # problem 1: rank j now has both
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"])
    assert (iters == 60).all()
    for b in range(B):
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(SWEEP_TIERS), plan[b], iters[b], err[b], 60, 0.0)
    assert plan[1][j, j] > 0                             # the diagonal entry took part
    pl.close()


def test_tiered_kernel_with_two_tiers_only():
    """A node / cross-node cost without a rail-group tier is still a pure tier cost (the group and far tiers carry the
    same value): it takes the tier-by-tier sums, eight warps per problem, and the four-warp build for a large batch."""
    import paper_2608_03676_b200 as P
    R = 256
    C = W.cost_matrix(R, 8, (0.0, 1.0, 12.0), None)
    for B, check in ((6, 3), (600, 2)):
        pl = P.Planner(L=B, R=R, E=R, K=1, k=1, T=R, e2r=torch.arange(R, dtype=torch.int32), C=C, eps=1.2,
                       max_iters=80, tol=0.0)
        loads = W.sweep_rank_loads(B, R, seed=91, device="cuda")
        ex, sp, s, d = pl.excess_spare(loads)
        out = pl.sinkhorn(s, d)
        torch.cuda.synchronize()
        plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
        assert (iters == 80).all() and (info == 0).all()
        for b in range(check):
            check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 1.2, plan[b], iters[b], err[b], 80, 0.0)
        pl.close()


@pytest.mark.parametrize("R", [512, 1024])
def test_tiered_kernel_in_tolerance_mode_beyond_256_ranks(R):
    """The stopping rule of the eight-warp tier-by-tier kernel with 2 and 4 ranks per lane: first iterate whose row
    error meets the tolerance, or the cap."""
    B = 3
    pl, C = _planner(B, R, 0.1, iters=400, tol=1e-6)
    loads = W.sweep_rank_loads(B, R, seed=57, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    assert (iters >= 1).all() and (iters <= 400).all() and ((info & ~(2 | 16)) == 0).all()
    for b in range(B):
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(SWEEP_TIERS), plan[b], iters[b], err[b],
                               400, 1e-6)
    print(f"R={R}: iterations {iters.tolist()}")
    pl.close()


@pytest.mark.parametrize("R,B", [(256, 40), (256, 300), (256, 2400), (512, 300), (1024, 80)])
@pytest.mark.parametrize("tol", [0.0, 1e-6])
def test_tiered_kernel_builds_by_batch_size(R, B, tol):
    """The tier-by-tier kernel spreads a problem over eight, four or two warps depending on the batch (a problem
    alone on an SM; a batch that fills the GPU; the largest batches at 256 ranks) and on the rank count (1 to 8 ranks
    per lane): every build, with a fixed count and with the tolerance, sampled problems against the oracle."""
    import paper_2608_03676_b200 as P
    C = W.cost_matrix(R, 8, SWEEP_TIERS, 4)
    eps = 0.12 * max(SWEEP_TIERS)
    iters_cap = 60 if tol == 0.0 else 400
    pl = P.Planner(L=B, R=R, E=R, K=1, k=1, T=R, e2r=torch.arange(R, dtype=torch.int32), C=C, eps=eps,
                   max_iters=iters_cap, tol=tol)
    loads = W.sweep_rank_loads(B, R, seed=7 + R + B, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    iters, info = cpu(out["iters"]), cpu(out["info"])
    assert ((info & ~16) == 0).all(), info[info != 0]
    if tol == 0.0:
        assert (iters == iters_cap).all()
    else:
        assert (iters >= 1).all() and (iters < iters_cap).all(), (iters.min(), iters.max())
    s_h, d_h, err = cpu(s), cpu(d), cpu(out["row_err"])
    for b in sorted({0, B // 2, B - 1, int(iters.argmax()), int(iters.argmin())}):
        check_sinkhorn_problem(s_h[b], d_h[b], C.numpy(), eps, cpu(out["plan"][b]), iters[b], err[b], iters_cap, tol)
    # properties that hold for every problem, checked on the GPU
    tot = s.double().sum(1)
    col_viol = (out["plan"].double().sum(1) - d.double()).abs().sum(1)
    assert bool((col_viol <= 1e-5 * tot).all()) and bool((out["plan"] >= 0).all())
    pl.close()


@pytest.mark.parametrize("R,check_every", [(256, 1), (256, 5), (512, 3)])
def test_tiered_kernel_stops_at_the_first_checked_iterate_within_the_tolerance(R, check_every):
    """The eight-warp kernel learns that an iterate met the tolerance half a step late (a ninth warp sums the row
    error beside the iteration) and puts that iterate back: iteration count, plan and reported error must be those
    of the first CHECKED iterate within the tolerance, also when only every few iterates are checked.  eps is large
    enough for the problems to converge well before the cap."""
    import paper_2608_03676_b200 as P
    B = 6
    C = W.cost_matrix(R, 8, SWEEP_TIERS, 4)
    eps = 0.12 * max(SWEEP_TIERS)
    pl = P.Planner(L=B, R=R, E=R, K=1, k=1, T=R, e2r=torch.arange(R, dtype=torch.int32), C=C, eps=eps,
                   max_iters=2000, tol=1e-6, check_every=check_every)
    loads = W.sweep_rank_loads(B, R, seed=91 + R, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    assert ((info & ~16) == 0).all(), info                       # nobody ran into the cap
    assert (iters < 2000).all() and (iters % check_every == 0).all(), iters
    for b in range(B):
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), eps, plan[b], iters[b], err[b], 2000, 1e-6, check_every)
    print(f"R={R} check_every={check_every}: iterations {iters.tolist()}")
    pl.close()


@pytest.mark.parametrize("R", [16, 64])
@pytest.mark.parametrize("B,check", [(1, 1), (4096, 6)])
@pytest.mark.parametrize("tol", [0.0, 1e-6])
def test_smallest_and_largest_batch_of_the_sweep(R, B, check, tol):
    """The two ends of the sweep's batch axis (one problem; 4096 problems, the register-capped batch builds of the
    one-warp kernels), with a fixed count and in tolerance mode, sampled problems against the oracle."""
    iters_cap = 300
    pl, C = _planner(B, R, 0.1, iters=iters_cap, tol=tol)
    loads = W.sweep_rank_loads(B, R, seed=2000 + R + B, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    if tol > 0:
        assert (iters >= 1).all() and (iters <= iters_cap).all() and ((info & ~2) == 0).all()
    else:
        assert (iters == iters_cap).all() and (info == 0).all()
    sample = sorted(set([0, B - 1] + [int(x) for x in np.linspace(0, B - 1, check)]))
    if tol > 0 and B > 1:
        sample = sorted(set(sample + [int(iters.argmax()), int(iters.argmin())]))
    for b in sample:
        check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(SWEEP_TIERS), plan[b], iters[b], err[b],
                               iters_cap, tol)
    tot = s.double().sum(1)
    col_viol = (out["plan"].double().sum(1) - d.double()).abs().sum(1)
    assert bool((col_viol <= 1e-5 * tot).all()) and bool((out["plan"] >= 0).all())
    pl.close()


@pytest.mark.parametrize("R,B,iters,check", [(512, 300, 40, (0, 1, 299)), (1024, 256, 30, (0, 255)), (1024, 700, 12, (3, 699))])
def test_large_batch_with_a_general_cost_takes_the_tensor_core_solve(R, B, iters, check):
    """More than 256 ranks, a cost without tier structure, a fixed iteration count and a batch of 256 problems or more:
    the batch is solved as dense products on the tensor cores (three TF32 products per term, four accumulators per
    tile).  Sampled problems against the oracle, a ragged last tile (B not a multiple of the tile width), and the
    marginals of every problem.  The tensor cores accumulate with truncation, so the row error this path reports -- the
    true row violation of the plan it returns -- may sit a few 1e-6 above the oracle's; it is held to the 1e-5 of total
    mass that bounds any marginal violation, the plan itself to the usual 1e-4 per entry."""
    from helpers import MASS_TOL
    pl, C = _planner(B, R, 0.1, iters=iters, general=True)
    loads = W.sweep_rank_loads(B, R, seed=4000 + R + B, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    assert pl.last_launch_count() == 2 * iters + 4          # prepare, two products per iteration, plan, report, input guard
    plan, it, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
    assert (it == iters).all() and (info == 0).all()
    for b in check:
        r = check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(SWEEP_TIERS), plan[b], it[b], err[b], iters,
                                   0.0, err_band=MASS_TOL)
        print(f"R={R} problem {b}: max rel err {r['max_rel']:.2e}")
    tot = s.double().sum(1)
    col_viol = (out["plan"].double().sum(1) - d.double()).abs().sum(1)
    assert bool((col_viol <= 1e-5 * tot).all()) and bool((out["plan"] >= 0).all())
    # the reported row error is the plan's own row violation
    row_viol = (out["plan"].double().sum(2) - s.double()).abs().sum(1) / tot
    assert bool(((row_viol - out["row_err"].double()).abs() <= 1e-6 + 1e-4 * row_viol).all())
    again = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    assert torch.equal(again["plan"], out["plan"]) and torch.equal(again["row_err"], out["row_err"])     # deterministic
    pl.close()


def test_tensor_core_solve_is_not_taken_where_it_does_not_apply():
    """Tolerance mode, a small batch or a Gibbs kernel near the edge of fp32 stay on the other kernels (launch counts
    tell which path ran); the results are checked by the cells above and by the sweep cells."""
    R = 512
    for kw, B in ((dict(iters=30, tol=1e-6), 300), (dict(iters=30), 8)):
        pl, C = _planner(B, R, 0.1, general=True, **kw)
        loads = W.sweep_rank_loads(B, R, seed=9, device="cuda")
        ex, sp, s, d = pl.excess_spare(loads)
        pl.sinkhorn(s, d)
        torch.cuda.synchronize()
        assert pl.last_launch_count() <= 4
        pl.close()
    pl, C = _planner(300, R, 0.01, iters=30, general=True)      # C / eps up to 100: beyond the range the dense form is built for
    loads = W.sweep_rank_loads(300, R, seed=9, device="cuda")
    ex, sp, s, d = pl.excess_spare(loads)
    out = pl.sinkhorn(s, d)
    torch.cuda.synchronize()
    assert pl.last_launch_count() <= 4
    check_sinkhorn_problem(cpu(s)[0], cpu(d)[0], C.numpy(), 0.01 * max(SWEEP_TIERS), cpu(out["plan"])[0], cpu(out["iters"])[0],
                           cpu(out["row_err"])[0], 30, 0.0)
    pl.close()


@pytest.mark.parametrize("gpus_per_node,nodes_per_group,want", [(4, 4, (4, 16)), (4, 8, (4, 32)), (16, 2, (16, 32)), (8, 4, (8, 32)),
                                                                (2, 4, (0, 0))])
def test_hierarchies_other_than_8_gpus_per_node_are_found_in_the_cost_matrix(gpus_per_node, nodes_per_group, want):
    """The tier-by-tier kernels are chosen from the cost matrix itself: 4- and 16-GPU nodes at 256 ranks take them too
    (a shape that is not built, 2-GPU nodes here, takes the general kernels); every case against the oracle, few and many
    problems per call, and a two-tier cost."""
    import paper_2608_03676_b200 as P
    R = 256
    for tiers, npg in ((SWEEP_TIERS, nodes_per_group), ((0.0, 1.0, 9.0), None)):
        C = W.cost_matrix(R, gpus_per_node, tiers, npg)
        for B, check in ((5, 2), (600, 2)):
            pl = P.Planner(L=B, R=R, E=R, K=1, k=1, T=R, e2r=torch.arange(R, dtype=torch.int32), C=C, eps=0.1 * max(tiers),
                           max_iters=60, tol=0.0)
            found = pl.tier_structure()
            if npg is not None:
                assert found == want
            else:
                assert found == ((gpus_per_node, 32) if gpus_per_node in (4, 8, 16) else (0, 0))
            loads = W.sweep_rank_loads(B, R, seed=300 + gpus_per_node, device="cuda")
            ex, sp, s, d = pl.excess_spare(loads)
            out = pl.sinkhorn(s, d)
            torch.cuda.synchronize()
            plan, iters, err, info = cpu(out["plan"]), cpu(out["iters"]), cpu(out["row_err"]), cpu(out["info"])
            assert (iters == 60).all() and (info == 0).all()
            for b in range(check):
                check_sinkhorn_problem(cpu(s)[b], cpu(d)[b], C.numpy(), 0.1 * max(tiers), plan[b], iters[b], err[b], 60, 0.0)
            pl.close()
