"""numpy wrappers around the C oracle (test infrastructure only)."""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "taot_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no FMA contraction, so fp32 scores round per operation)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-Wall",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_auction.restype = ctypes.c_int64
        _lib.oracle_sinkhorn.restype = ctypes.c_int32
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def histogram(topk: np.ndarray, R: int, E: int, e2r: np.ndarray):
    """topk int32 [L,T,k] -> n [L,R,E], expert_load [L,E], rank_load [L,R], bad [L]."""
    topk = _i32(topk)
    L, T, k = topk.shape
    e2r = _i32(e2r)
    n = np.empty((L, R, E), np.int32)
    el = np.empty((L, E), np.int32)
    rl = np.empty((L, R), np.int32)
    bad = np.empty((L,), np.int64)
    _L().oracle_histogram(_p(topk), ctypes.c_int32(L), ctypes.c_int64(T), ctypes.c_int32(k),
                          ctypes.c_int32(R), ctypes.c_int32(E), _p(e2r), _p(n), _p(el), _p(rl), _p(bad))
    return n, el, rl, bad


def excess_spare(rank_load: np.ndarray):
    """rank_load int32 [L,R] -> mean int64 [L], excess int32 [L,R], spare int32 [L,R]."""
    rl = _i32(rank_load)
    L, R = rl.shape
    mean = np.empty((L,), np.int64)
    ex = np.empty((L, R), np.int32)
    sp = np.empty((L, R), np.int32)
    _L().oracle_excess_spare(_p(rl), ctypes.c_int32(L), ctypes.c_int32(R), _p(mean), _p(ex), _p(sp))
    return mean, ex, sp


def sinkhorn(s, d, C, eps: float, max_iters: int, tol: float = 0.0, check_every: int = 1,
             eps0: float = 1e-8, history: bool = False):
    """One problem.  s, d fp32 [R]; C fp32 [R,R].  Returns dict(plan fp64 [R,R], n_iter, row_err,
    capped, err_hist)."""
    s = _f32(s); d = _f32(d); C = _f32(C)
    R = s.shape[0]
    plan = np.empty((R, R), np.float64)
    n_iter = ctypes.c_int32(0)
    row_err = ctypes.c_double(0.0)
    hist = np.full((max(max_iters, 1),), np.nan, np.float64) if history else None
    st = _L().oracle_sinkhorn(_p(s), _p(d), ctypes.c_int32(R), _p(C), ctypes.c_float(eps),
                              ctypes.c_float(eps0), ctypes.c_int32(max_iters), ctypes.c_double(tol),
                              ctypes.c_int32(max(1, check_every)), _p(plan), ctypes.byref(n_iter),
                              ctypes.byref(row_err), _p(hist))
    return dict(plan=plan, n_iter=int(n_iter.value), row_err=float(row_err.value), capped=bool(st),
                err_hist=None if hist is None else hist[: n_iter.value])


def sinkhorn_gibbs(s, d, C, eps: float, iters: int, eps0: float = 1e-8) -> np.ndarray:
    s = _f32(s); d = _f32(d); C = _f32(C)
    R = s.shape[0]
    plan = np.empty((R, R), np.float64)
    _L().oracle_sinkhorn_gibbs(_p(s), _p(d), ctypes.c_int32(R), _p(C), ctypes.c_float(eps),
                               ctypes.c_float(eps0), ctypes.c_int32(iters), _p(plan))
    return plan


def default_preference(C) -> np.ndarray:
    C = _f32(C)
    R = C.shape[0]
    B = np.empty((R, R), np.float32)
    _L().oracle_default_preference(_p(C), ctypes.c_int32(R), _p(B))
    return B


def spill(expert_load, e2r, R: int, mean: int) -> np.ndarray:
    el = _i32(expert_load); e2r = _i32(e2r)
    E = el.shape[0]
    out = np.empty((E,), np.int32)
    _L().oracle_spill(_p(el), _p(e2r), ctypes.c_int32(R), ctypes.c_int32(E), ctypes.c_int64(int(mean)), _p(out))
    return out


def match(R: int, E: int, K: int, e2r, mean: int, excess, spill_in, spare_in, B, plan32, eps0: float = 1e-8):
    """Phase 2 for one layer.  Returns dict(slot_expert [R*K], slot_tokens [R*K], spill_left, spare_left,
    inner_rounds)."""
    e2r = _i32(e2r); excess = _i32(excess)
    sp = _i32(spill_in).copy(); sr = _i32(spare_in).copy()
    B = _f32(B); plan32 = _f32(plan32)
    se = np.empty((R * K,), np.int32)
    stk = np.empty((R * K,), np.int32)
    rounds = ctypes.c_int32(0)
    _L().oracle_match(ctypes.c_int32(R), ctypes.c_int32(E), ctypes.c_int32(K), _p(e2r),
                      ctypes.c_int64(int(mean)), _p(excess), _p(sp), _p(sr), _p(B), _p(plan32),
                      ctypes.c_float(eps0), _p(se), _p(stk), ctypes.byref(rounds))
    return dict(slot_expert=se, slot_tokens=stk, spill_left=sp, spare_left=sr, inner_rounds=int(rounds.value))


def auction(R: int, E: int, K: int, n, slot_expert, slot_tokens, B, price_step: float = 0.1,
            max_rounds: int = 0):
    """Phase 3 for one layer.  n int32 [R,E].  Returns dict(X [R,S], rounds, residual)."""
    n = _i32(n); se = _i32(slot_expert); stk = _i32(slot_tokens); B = _f32(B)
    S = R * K
    X = np.empty((R, S), np.int32)
    rounds = ctypes.c_int32(0)
    res = _L().oracle_auction(ctypes.c_int32(R), ctypes.c_int32(E), ctypes.c_int32(K), _p(n), _p(se),
                              _p(stk), _p(B), ctypes.c_float(price_step), ctypes.c_int32(max_rounds),
                              _p(X), ctypes.byref(rounds))
    return dict(X=X, rounds=int(rounds.value), residual=int(res))


def assign(topk_layer, R: int, E: int, K: int, slot_expert, X) -> np.ndarray:
    """Token reassignment for one layer.  topk_layer int32 [T,k] -> new_idx int32 [T,k]."""
    topk = _i32(topk_layer)
    T, k = topk.shape
    se = _i32(slot_expert); X = _i32(X)
    out = np.empty((T, k), np.int32)
    _L().oracle_assign(_p(topk), ctypes.c_int64(T), ctypes.c_int32(k), ctypes.c_int32(R),
                       ctypes.c_int32(E), ctypes.c_int32(K), _p(se), _p(X), _p(out))
    return out


def dispatch(new_idx_layer, R: int, E: int, K: int, e2r):
    """Dispatch metadata of one rewritten routing table (the step after the planner: what the token
    all-to-all needs).  new_idx_layer int32 [T,k]: e in [0,E) = expert e on its home rank, E + s = guest slot
    s on rank s // K.  Source rank r owns the R contiguous segments of T/R*k entries.

    Definition, per source rank: order its entries by (destination rank, target index) keeping the original
    flat order among equal keys (a stable sort); perm[i] is the position of entry i in that order, i.e. its
    place in the rank's send buffer.  send_counts[r][q] = entries of source rank r that execute on rank q;
    target_counts[r][t] = entries of source rank r with target t (t < E + S).  An index outside [0, E + S)
    cannot be delivered: it is counted nowhere and sorts after every valid entry, in its original order.

    Returns dict(perm int32 [T,k], send_counts int32 [R,R], target_counts int32 [R,E+S], bad int)."""
    x = _i32(new_idx_layer)
    T, k = x.shape
    S = R * K
    e2r = _i32(e2r).astype(np.int64)
    seg = T // R * k
    flat = x.reshape(R, seg).astype(np.int64)
    valid = (flat >= 0) & (flat < E + S)
    safe = np.where(valid, flat, 0)
    dest = np.where(safe < E, e2r[np.minimum(safe, E - 1)], (safe - E) // K)
    key = np.where(valid, dest * (E + S) + safe, R * (E + S))
    perm = np.empty((R, seg), np.int32)
    send = np.zeros((R, R), np.int32)
    tc = np.zeros((R, E + S), np.int32)
    for r in range(R):
        order = np.argsort(key[r], kind="stable")
        perm[r, order] = np.arange(seg, dtype=np.int32)
        send[r] = np.bincount(dest[r][valid[r]], minlength=R)
        tc[r] = np.bincount(flat[r][valid[r]], minlength=E + S)
    return dict(perm=perm.reshape(T, k), send_counts=send, target_counts=tc, bad=int((~valid).sum()))


REPORT_INTS = ("total_load", "rerouted", "mean_load", "max_before", "min_before", "max_after", "min_after",
               "hot_ranks", "cold_ranks", "hot_experts", "clones", "intra", "inter", "same_rank")
REPORT_REALS = ("rho_before", "rho_after", "dev_before", "dev_after", "peak_reduction", "frac_rerouted",
                "cost_ratio", "cost_C")


def report(R: int, E: int, K: int, e2r, C, B, expert_load, rank_load, slot_expert, X, lam: float = 3.0):
    """Dispatch report of one layer.  Returns a dict with the scalar fields named in REPORT_INTS /
    REPORT_REALS and the arrays spill [E], load_after [R], slot_moved [S], slot_kind [S]."""
    e2r = _i32(e2r); C = _f32(C); B = _f32(B)
    el = _i32(expert_load); rl = _i32(rank_load); se = _i32(slot_expert).reshape(-1); X = _i32(X)
    S = R * K
    spill_out = np.empty((E,), np.int32)
    la = np.empty((R,), np.int32)
    moved = np.empty((S,), np.int32)
    kind = np.empty((S,), np.int32)
    ints = np.zeros((len(REPORT_INTS),), np.int64)
    reals = np.zeros((len(REPORT_REALS),), np.float64)
    _L().oracle_report(ctypes.c_int32(R), ctypes.c_int32(E), ctypes.c_int32(K), _p(e2r), _p(C), _p(B),
                       _p(el), _p(rl), _p(se), _p(X), ctypes.c_double(lam), _p(spill_out), _p(la),
                       _p(moved), _p(kind), _p(ints), _p(reals))
    out = dict(spill=spill_out, load_after=la, slot_moved=moved, slot_kind=kind)
    out.update({k: int(v) for k, v in zip(REPORT_INTS, ints)})
    out.update({k: float(v) for k, v in zip(REPORT_REALS, reals)})
    return out


def plan_layers(topk, R: int, E: int, K: int, e2r, C, eps: float, max_iters: int, tol: float = 0.0,
                check_every: int = 1, B=None, eps0: float = 1e-8, price_step: float = 0.1,
                auction_max_rounds: int = 0, do_assign: bool = True, hint: bool = True,
                topology: bool = True):
    """The whole path on the CPU, layer by layer: histogram, excess/spare, Sinkhorn (the fp64 plan
    is rounded to fp32 before it is used as the Phase-2 hint, as the library's plan is fp32),
    spill, matching, auction, reassignment.

    The two switches of the paper's ablation (Ablation Study, Table 2): hint=False leaves the
    Phase-1 term out of the Phase-2 score (Phase 1 is not run, the plan is zero); topology=False
    leaves the topology-preference term out of the Phase-2 score.  A term left out is a term that
    is exactly zero, so the matching is fed a zero plan / a zero preference matrix.  Phase 3 is not
    ablated and always sees the real preference matrix."""
    topk = _i32(topk)
    L = topk.shape[0]
    C = _f32(C)
    Bm = default_preference(C) if B is None else _f32(B)
    n, el, rl, bad = histogram(topk, R, E, e2r)
    mean, ex, sp = excess_spare(rl)
    out = dict(n=n, expert_load=el, rank_load=rl, bad=bad, mean=mean, excess=ex, spare=sp,
               plan=np.zeros((L, R, R), np.float64), n_iter=np.zeros(L, np.int32),
               row_err=np.zeros(L), slot_expert=np.zeros((L, R, K), np.int32),
               slot_tokens=np.zeros((L, R, K), np.int32), X=np.zeros((L, R, R * K), np.int32),
               auction_rounds=np.zeros(L, np.int32), match_rounds=np.zeros(L, np.int32),
               new_idx=np.empty_like(topk) if do_assign else None)
    B2 = Bm if topology else np.zeros_like(Bm)
    for l in range(L):
        if hint:
            sk = sinkhorn(ex[l].astype(np.float32), sp[l].astype(np.float32), C, eps, max_iters, tol,
                          check_every, eps0)
            out["plan"][l] = sk["plan"]; out["n_iter"][l] = sk["n_iter"]; out["row_err"][l] = sk["row_err"]
        spl = spill(el[l], e2r, R, mean[l])
        m = match(R, E, K, e2r, mean[l], ex[l], spl, sp[l], B2, out["plan"][l].astype(np.float32), eps0)
        out["slot_expert"][l] = m["slot_expert"].reshape(R, K)
        out["slot_tokens"][l] = m["slot_tokens"].reshape(R, K)
        out["match_rounds"][l] = m["inner_rounds"]
        a = auction(R, E, K, n[l], m["slot_expert"], m["slot_tokens"], Bm, price_step, auction_max_rounds)
        out["X"][l] = a["X"]; out["auction_rounds"][l] = a["rounds"]
        if do_assign:
            out["new_idx"][l] = assign(topk[l], R, E, K, m["slot_expert"], a["X"])
    return out
