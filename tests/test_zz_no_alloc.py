"""`taot_histogram_static`: load collection for callers that cannot allocate device memory (a
plug-in inside a runtime that owns all device memory, a stage of a captured step).  It keeps its
per-chunk counts in a fixed array inside the library instead of a caller workspace.  Checked here,
through the C ABI, against `taot_histogram` on two calls in a row that share that array: a larger
problem first, then a smaller one with different data, so stale counts from the first call would
show.  Integer outputs: bit-exact.  This file is named to be collected last."""
import pytest
import torch

import oracle as O
import workloads as W

pytestmark = pytest.mark.gpu


def _both(cfg):
    import paper_2608_03676_b200 as P
    topk = W.routing_topk(cfg, device="cuda")
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode)
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group)
    pl = P.Planner(L=cfg.L, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r, C=C, eps=cfg.eps,
                   max_iters=cfg.max_iters, tol=cfg.tol)
    want = pl.histogram(topk)                                   # the existing entry point (workspace-based)
    # everything the no-allocation call touches is allocated before it, by the caller
    e2r_dev = e2r.cuda()
    n = torch.full((cfg.L, cfg.R, cfg.E), -7, dtype=torch.int32, device="cuda")
    el = torch.full((cfg.L, cfg.E), -7, dtype=torch.int32, device="cuda")
    rl = torch.full((cfg.L, cfg.R), -7, dtype=torch.int32, device="cuda")
    info = torch.zeros((cfg.L,), dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    rc = P.histogram_static(topk, cfg.R, cfg.E, e2r_dev, n, el, rl, info)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before              # torch's allocator was not asked for anything
    assert rc == 0
    assert torch.equal(n, want[0]) and torch.equal(el, want[1]) and torch.equal(rl, want[2])
    assert int(info.abs().sum()) == 0
    assert int(n.sum()) == cfg.L * cfg.T * cfg.k
    # and directly against the CPU oracle's definition of the loads
    n_o, el_o, rl_o, bad_o = O.histogram(topk.cpu().numpy(), cfg.R, cfg.E, e2r.numpy())
    assert (n.cpu().numpy() == n_o).all() and (el.cpu().numpy() == el_o).all() and (rl.cpu().numpy() == rl_o).all()
    assert (bad_o == 0).all()
    pl.close()


def test_static_histogram_matches_workspace_histogram_on_two_calls_in_a_row():
    # 24 x 16 x 2 chunks x 64 experts of counts (a ragged second chunk), then a smaller, different problem
    _both(W.get_config("cfg2").replace(T=16 * 2560))
    _both(W.get_config("cfg1"))
    _both(W.get_config("cfg2").replace(L=3, seed=99))


def test_static_histogram_rejects_what_does_not_fit():
    import paper_2608_03676_b200 as P
    cfg = W.get_config("cfg3").replace(L=58, T=64 * 4096)       # 58*64*2*256*4 B = 7.6 MB > 4 MiB
    topk = torch.zeros((cfg.L, cfg.T, cfg.k), dtype=torch.int32, device="cuda")
    e2r_dev = W.expert_to_rank(cfg.E, cfg.R).cuda()
    n = torch.full((cfg.L, cfg.R, cfg.E), -7, dtype=torch.int32, device="cuda")
    el = torch.zeros((cfg.L, cfg.E), dtype=torch.int32, device="cuda")
    rl = torch.zeros((cfg.L, cfg.R), dtype=torch.int32, device="cuda")
    info = torch.zeros((cfg.L,), dtype=torch.int32, device="cuda")
    rc = P.histogram_static(topk, cfg.R, cfg.E, e2r_dev, n, el, rl, info)
    torch.cuda.synchronize()
    assert rc == -6
    assert b"TAOT_STATIC_SCRATCH_BYTES" in P.load_library().taot_status_string(rc)
    assert int((n != -7).sum()) == 0                            # nothing was launched


def test_static_histogram_flags_a_home_rank_out_of_range_instead_of_writing_out_of_bounds():
    """The expert-to-rank map is the caller's device memory here and nobody validated it: an entry outside
    [0, R) must be caught on the device (flag, expert left out of the rank loads), not used as an address."""
    import paper_2608_03676_b200 as P
    cfg = W.get_config("cfg2").replace(L=2)
    topk = W.routing_topk(cfg, device="cuda")
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode)
    bad = e2r.clone(); bad[7] = cfg.R + 1000; bad[20] = -3
    n = torch.zeros((cfg.L, cfg.R, cfg.E), dtype=torch.int32, device="cuda")
    el = torch.zeros((cfg.L, cfg.E), dtype=torch.int32, device="cuda")
    rl = torch.zeros((cfg.L, cfg.R), dtype=torch.int32, device="cuda")
    info = torch.zeros((cfg.L,), dtype=torch.int32, device="cuda")
    rc = P.histogram_static(topk, cfg.R, cfg.E, bad.cuda(), n, el, rl, info)
    torch.cuda.synchronize()
    assert rc == 0 and bool((info & P.INFO_BAD_INDEX).bool().all())
    n_o, el_o, rl_o, _ = O.histogram(topk.cpu().numpy(), cfg.R, cfg.E, e2r.numpy())
    assert (n.cpu().numpy() == n_o).all() and (el.cpu().numpy() == el_o).all()       # counts do not depend on the map
    want = rl_o.copy()
    want[:, int(e2r[7])] -= el_o[:, 7]; want[:, int(e2r[20])] -= el_o[:, 20]                   # the two experts are left out
    assert (rl.cpu().numpy() == want).all()
