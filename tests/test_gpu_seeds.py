"""Other seeds and shapes through the whole planner: every stage of `taot_plan` against the oracle, as in the edge
tests, on routing tables the other tests do not use (the seeded generator draws different experts, hot experts and
permutations, so quota intervals, cursor walks and split chunks fall elsewhere)."""
import pytest

import workloads as W
from helpers import make_planner
from test_gpu_edge import _full_check

pytestmark = pytest.mark.gpu

SHAPES = {
    "cfg4_two_chunks_ragged": ("cfg4", dict(L=2, T=256 * 2304)),      # 256 ranks: tiered Sinkhorn, bit-set auction
    "cfg4_two_slots_per_rank": ("cfg4", dict(L=2, T=256 * 4096, K=2)),
    "cfg4_four_slots_per_rank": ("cfg4", dict(L=1, T=256 * 2048, K=4)),  # 1024 slots: every thread of the CTA holds one
    "cfg3_ragged": ("cfg3", dict(L=3, T=64 * 2560)),
    "cfg3_four_chunks": ("cfg3", dict(L=2, T=64 * 8192)),
    "cfg2": ("cfg2", dict(L=4)),
}


@pytest.mark.parametrize("shape", sorted(SHAPES))
@pytest.mark.parametrize("seed", [11, 37])
def test_full_path_on_other_seeds(shape, seed):
    name, over = SHAPES[shape]
    cfg = W.get_config(name)
    cfg = cfg.replace(seed=cfg.seed + seed, **over)
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg)
    _full_check(cfg, topk, pl)
    pl.close()
