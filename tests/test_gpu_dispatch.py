"""GPU parity of the dispatch metadata (send counts, target counts, stable send-buffer positions)
against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from helpers import cpu, make_planner, topology

pytestmark = pytest.mark.gpu

CASES = {
    "cfg1": W.get_config("cfg1"),
    "cfg2": W.get_config("cfg2").replace(L=4),
    "cfg3_small": W.get_config("cfg3").replace(L=2, T=64 * 2560),       # 2 chunks per segment, ragged
    "cfg4_small": W.get_config("cfg4").replace(L=2, T=256 * 2304),
    "ladder32": W.get_config("ladder32").replace(L=3),
    "ragged": W.get_config("cfg1").replace(L=2, T=8 * 1237, k=3),       # segment of 3711 entries: partial warps
}


@pytest.mark.parametrize("name", list(CASES))
def test_dispatch_bit_exact(name):
    cfg = CASES[name]
    e2r, _ = topology(cfg)
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg)
    out = pl.plan(topk)
    d = pl.dispatch(out["new_idx"])
    torch.cuda.synchronize()
    assert pl.last_launch_count() == 3
    new = cpu(out["new_idx"])
    for l in range(cfg.L):
        want = O.dispatch(new[l], cfg.R, cfg.E, cfg.K, e2r.numpy())
        assert (cpu(d["send_counts"])[l] == want["send_counts"]).all()
        assert (cpu(d["target_counts"])[l] == want["target_counts"]).all()
        assert (cpu(d["perm"])[l] == want["perm"]).all()
        assert cpu(d["info"])[l] == 0
    # what every rank receives is the projected load of the report
    rep = pl.report(out["expert_load"], out["rank_load"], out["slot_expert"], out["X"])
    assert (cpu(d["send_counts"]).sum(1) == cpu(rep["load_after"])).all()
    # deterministic, and the optional output may be skipped
    d2 = pl.dispatch(out["new_idx"], want_target_counts=False)
    assert (cpu(d2["perm"]) == cpu(d["perm"])).all() and d2["target_counts"] is None
    pl.close()


def test_dispatch_undeliverable_indices_and_errors():
    import ctypes
    cfg = W.get_config("cfg1").replace(L=2)
    e2r, _ = topology(cfg)
    topk = W.routing_topk(cfg, device="cuda")
    pl = make_planner(cfg)
    new = pl.plan(topk)["new_idx"].clone()
    g = torch.Generator(device="cuda").manual_seed(3)
    hit = torch.rand(new.shape, generator=g, device="cuda") < 0.01
    new[hit] = torch.where(torch.rand(new.shape, generator=g, device="cuda")[hit] < 0.5, -7, cfg.E + cfg.S + 5).int()
    new[1] = torch.clamp(new[1], 0, cfg.E + cfg.S - 1)              # layer 1 stays clean
    d = pl.dispatch(new)
    torch.cuda.synchronize()
    for l in range(cfg.L):
        want = O.dispatch(cpu(new)[l], cfg.R, cfg.E, cfg.K, e2r.numpy())
        assert (cpu(d["perm"])[l] == want["perm"]).all() and (cpu(d["send_counts"])[l] == want["send_counts"]).all()
        assert bool(cpu(d["info"])[l] & 1) == (want["bad"] > 0)
    assert cpu(d["info"]).tolist()[1] == 0 and cpu(d["info"]).tolist()[0] == 1
    ptr = lambda t: ctypes.c_void_p(t.data_ptr())
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    send = torch.empty((cfg.L, cfg.R, cfg.R), dtype=torch.int32, device="cuda")
    info = torch.zeros(cfg.L, dtype=torch.int32, device="cuda")
    assert pl.lib.taot_dispatch(pl.handle, ptr(new), ptr(send), None, ptr(new), ptr(info), ptr(pl.ws), st) == -2
    assert pl.lib.taot_dispatch(pl.handle, ptr(new), None, None, ptr(send), ptr(info), ptr(pl.ws), st) == -1
    pl.close()
