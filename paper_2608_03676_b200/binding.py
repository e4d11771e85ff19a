"""ctypes binding of include/taot.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Dict, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libtaot.so")
_lib = None

INFO_BAD_INDEX = 1
INFO_SINKHORN_CAP = 2
INFO_NONFINITE = 4
INFO_AUCTION_RESIDUAL = 8
INFO_SUPPLY_SCALED = 16
INFO_SINKHORN_SIZE = 32
INFO_INTERNAL = 64

ABLATE_HINT = 1
ABLATE_TOPOLOGY = 2

_SYMBOLS = [
    "taot_create", "taot_destroy", "taot_workspace_bytes", "taot_host_workspace_bytes",
    "taot_histogram", "taot_histogram_static", "taot_excess_spare", "taot_sinkhorn", "taot_match", "taot_assign",
    "taot_plan", "taot_plan_host", "taot_host_block_layout", "taot_plan_host_block", "taot_report", "taot_dispatch", "taot_measure_alu_peaks", "taot_measure_latencies", "taot_measure_round_latencies", "taot_set_profiling", "taot_get_stage_ms", "taot_get_match_cycles", "taot_get_group_trace", "taot_tier_structure", "taot_last_launch_count",
    "taot_status_string",
]


class TaotError(RuntimeError):
    pass


class TaotParams(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_int32), ("L", ctypes.c_int32), ("R", ctypes.c_int32),
        ("E", ctypes.c_int32), ("K", ctypes.c_int32), ("k", ctypes.c_int32), ("T", ctypes.c_int64),
        ("eps", ctypes.c_float), ("max_iters", ctypes.c_int32), ("tol", ctypes.c_float),
        ("check_every", ctypes.c_int32), ("eps0", ctypes.c_float), ("price_step", ctypes.c_float),
        ("auction_max_rounds", ctypes.c_int32), ("ablation", ctypes.c_int32),
    ]


class ReportRow(ctypes.Structure):
    """taot_report_row: one layer's dispatch diagnostics (128 bytes)."""
    _fields_ = [
        ("total_load", ctypes.c_int64), ("rerouted", ctypes.c_int64), ("mean_load", ctypes.c_int32),
        ("max_before", ctypes.c_int32), ("min_before", ctypes.c_int32), ("max_after", ctypes.c_int32),
        ("min_after", ctypes.c_int32), ("hot_ranks", ctypes.c_int32), ("cold_ranks", ctypes.c_int32),
        ("hot_experts", ctypes.c_int32), ("clones", ctypes.c_int32), ("intra", ctypes.c_int32),
        ("inter", ctypes.c_int32), ("same_rank", ctypes.c_int32),
        ("rho_before", ctypes.c_double), ("rho_after", ctypes.c_double), ("dev_before", ctypes.c_double),
        ("dev_after", ctypes.c_double), ("peak_reduction", ctypes.c_double), ("frac_rerouted", ctypes.c_double),
        ("cost_ratio", ctypes.c_double), ("cost_C", ctypes.c_double),
    ]


class _Outputs(ctypes.Structure):
    _fields_ = [(name, ctypes.c_void_p) for name in (
        "n", "expert_load", "rank_load", "excess", "spare", "plan", "sinkhorn_iters", "row_err",
        "slot_expert", "slot_tokens", "X", "rounds", "new_idx", "info")]


def library_path() -> str:
    return _LIB_PATH


def exported_symbols():
    return list(_SYMBOLS)


def load_library() -> ctypes.CDLL:
    """Load libtaot.so; raise if it has not been built (there is no other code path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise TaotError(f"{_LIB_PATH} is missing: build it with `python -m paper_2608_03676_b200.build`")
        lib = ctypes.CDLL(_LIB_PATH)
        for name in _SYMBOLS:
            getattr(lib, name)                      # raises AttributeError if a symbol is absent
        lib.taot_status_string.restype = ctypes.c_char_p
        for name in _SYMBOLS:
            if name != "taot_status_string":
                getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        msg = load_library().taot_status_string(rc).decode()
        raise TaotError(f"{what}: {msg} ({rc})")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TaotError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


STATIC_SCRATCH_BYTES = 4 << 20
# kernels one taot_plan call enqueues: chunk histogram, merge, Sinkhorn (register tile + shared-memory
# kernel for handed-back problems), matching+auction, reassignment (a handle that splits a 256-rank table into layer
# groups adds one launch per group: the one-byte copy of the group's table)
PLAN_LAUNCHES = 6
PLAN_LAUNCHES_NO_HINT = 4       # with ABLATE_HINT the two Sinkhorn kernels are not launched


def histogram_static(topk: torch.Tensor, R: int, E: int, e2r_dev: torch.Tensor, n: torch.Tensor,
                     expert_load: torch.Tensor, rank_load: torch.Tensor, info: torch.Tensor) -> int:
    """Load collection through `taot_histogram_static`, the entry point for callers that cannot
    allocate device memory: no handle, no workspace; the caller passes every input and output
    (CUDA tensors it already owns) and gets the status code back instead of an exception, so that
    a caller in a no-allocation region can decide what to do.  Problems whose per-chunk counts
    exceed STATIC_SCRATCH_BYTES return the capacity error (-6) and launch nothing.  Calls share one
    built-in scratch array per GPU: do not let two of them overlap on the device."""
    lib = load_library()
    L, T, k = topk.shape
    for t, dt, nm in ((topk, torch.int32, "topk"), (e2r_dev, torch.int32, "e2r"), (n, torch.int32, "n"),
                      (expert_load, torch.int32, "expert_load"), (rank_load, torch.int32, "rank_load"),
                      (info, torch.int32, "info")):
        _dev(t, dt, nm)
    return int(lib.taot_histogram_static(_ptr(topk), ctypes.c_int32(L), ctypes.c_int64(T), ctypes.c_int32(k),
                                         ctypes.c_int32(R), ctypes.c_int32(E), _ptr(e2r_dev), _ptr(n),
                                         _ptr(expert_load), _ptr(rank_load), _ptr(info), _stream()))


def measure_alu_peaks() -> Dict[str, float]:
    """FP32-FMA (TFLOP/s) and ex2 (T op/s) throughput of the current GPU, measured by `taot_measure_alu_peaks`."""
    lib = load_library()
    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    sink = torch.zeros(2048 * sms, dtype=torch.float32, device="cuda")
    fma = ctypes.c_float(); ex2 = ctypes.c_float()
    _check(lib.taot_measure_alu_peaks(ctypes.byref(fma), ctypes.byref(ex2), _ptr(sink), _stream()),
           "taot_measure_alu_peaks")
    return dict(fma_tflops=float(fma.value), ex2_tops=float(ex2.value))


def measure_latencies() -> Dict[str, float]:
    """SM clock cycles per dependent operation on the current GPU (`taot_measure_latencies`): one shuffle-reduction
    level, one FMA, one reciprocal-and-multiply."""
    lib = load_library()
    sink = torch.zeros(4, dtype=torch.float32, device="cuda")
    cyc = (ctypes.c_float * 3)()
    _check(lib.taot_measure_latencies(cyc, _ptr(sink), _stream()), "taot_measure_latencies")
    return dict(shuffle_level=float(cyc[0]), fma=float(cyc[1]), rcp_mul=float(cyc[2]))


def measure_round_latencies() -> Dict[str, float]:
    """SM clock cycles of the operations an auction round is a chain of (`taot_measure_round_latencies`): a dependent
    shared-memory load, a shared-memory atomicMax waited for, a named barrier over eight warps, and the arbitration
    triple (atomicMax, barrier, read-back) as a unit."""
    lib = load_library()
    sink = torch.zeros(8, dtype=torch.float32, device="cuda")
    cyc = (ctypes.c_float * 4)()
    _check(lib.taot_measure_round_latencies(cyc, _ptr(sink), _stream()), "taot_measure_round_latencies")
    return dict(shared_load=float(cyc[0]), shared_atomic=float(cyc[1]), barrier=float(cyc[2]), arbitration=float(cyc[3]))


@dataclass
class PlanResult:
    tensors: Dict[str, torch.Tensor]

    def __getitem__(self, key):
        return self.tensors[key]


class Planner:
    """One planner handle for a fixed topology (e2r, C, optional B) and problem shape."""

    def __init__(self, L: int, R: int, E: int, K: int, k: int, T: int, e2r, C, eps: float,
                 max_iters: int, tol: float = 0.0, check_every: int = 1, B=None, eps0: float = 1e-8,
                 price_step: float = 0.1, auction_max_rounds: int = 0, ablation: int = 0,
                 device: Optional[torch.device] = None):
        if not torch.cuda.is_available():
            raise TaotError("the TAOT planner needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.L, self.R, self.E, self.K, self.k, self.T = L, R, E, K, k, T
        self.S = R * K
        p = TaotParams(ctypes.sizeof(TaotParams), L, R, E, K, k, T, eps, max_iters, tol, check_every, eps0,
                       price_step, auction_max_rounds, ablation)
        self.params = p
        self.ablation = ablation
        e2r_h = torch.as_tensor(e2r, dtype=torch.int32).contiguous().cpu()
        C_h = torch.as_tensor(C, dtype=torch.float32).contiguous().cpu()
        B_h = None if B is None else torch.as_tensor(B, dtype=torch.float32).contiguous().cpu()
        if e2r_h.numel() != E or C_h.numel() != R * R or (B_h is not None and B_h.numel() != R * R):
            raise TaotError("e2r / C / B have the wrong number of elements")
        self.handle = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.taot_create(ctypes.byref(self.handle), ctypes.byref(p), _ptr(e2r_h), _ptr(C_h),
                                        _ptr(B_h)), "taot_create")
            n = ctypes.c_size_t()
            _check(self.lib.taot_workspace_bytes(self.handle, ctypes.byref(n)), "taot_workspace_bytes")
            self.ws_bytes = n.value
            _check(self.lib.taot_host_workspace_bytes(self.handle, ctypes.byref(n)), "taot_host_workspace_bytes")
            self.host_ws_bytes = n.value
            self.ws = torch.empty(max(self.ws_bytes, 256), dtype=torch.uint8, device=self.device)
        self._host_ws = None

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle.value:
            self.lib.taot_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ allocation helpers
    def _empty(self, shape, dtype):
        return torch.empty(shape, dtype=dtype, device=self.device)

    def alloc_outputs(self) -> Dict[str, torch.Tensor]:
        L, R, E, K, S, T, k = self.L, self.R, self.E, self.K, self.S, self.T, self.k
        i32, f32 = torch.int32, torch.float32
        return dict(
            n=self._empty((L, R, E), i32), expert_load=self._empty((L, E), i32), rank_load=self._empty((L, R), i32),
            excess=self._empty((L, R), i32), spare=self._empty((L, R), i32), plan=self._empty((L, R, R), f32),
            sinkhorn_iters=self._empty((L,), i32), row_err=self._empty((L,), f32),
            slot_expert=self._empty((L, R, K), i32), slot_tokens=self._empty((L, R, K), i32),
            X=self._empty((L, R, S), i32), rounds=self._empty((L, 2), i32), new_idx=self._empty((L, T, k), i32),
            info=torch.zeros((L,), dtype=i32, device=self.device))

    def plan_launches(self) -> int:
        """Kernels one `plan` call of this handle enqueues when it plans all layers as one group; a handle that
        splits a large table into layer groups enqueues them once per group (`last_launch_count()` reports what the
        last call did)."""
        return PLAN_LAUNCHES_NO_HINT if (self.ablation & ABLATE_HINT) else PLAN_LAUNCHES

    def last_launch_count(self) -> int:
        c = ctypes.c_int32()
        _check(self.lib.taot_last_launch_count(self.handle, ctypes.byref(c)), "taot_last_launch_count")
        return c.value

    def set_profiling(self, on):
        """False / 0: off.  True / 1: stage events.  2: stage events and the cycle counters of the matching kernel."""
        _check(self.lib.taot_set_profiling(self.handle, ctypes.c_int32(int(on))), "taot_set_profiling")

    def stage_ms(self):
        """Durations (ms) of the five kernels of the last profiled plan call:
        chunk histogram, merge, Sinkhorn, matching+auction, reassignment.  Waits for them."""
        ms = (ctypes.c_float * 5)()
        _check(self.lib.taot_get_stage_ms(self.handle, ms), "taot_get_stage_ms")
        return [float(x) for x in ms]

    def tier_structure(self):
        """(ranks per node, ranks per rail group) of the hierarchy found in the cost matrix, or (0, 0) if the
        tier-by-tier Sinkhorn kernels do not apply to it."""
        n = ctypes.c_int32(0); g = ctypes.c_int32(0)
        _check(self.lib.taot_tier_structure(self.handle, ctypes.byref(n), ctypes.byref(g)), "taot_tier_structure")
        return n.value, g.value

    def group_trace(self):
        """Timeline (ms from the start of the call) of the layer groups of the last plan made with profiling level 3:
        a list with one [start, histogram, merge, Sinkhorn, matching, reassignment] row per group; [] if the handle
        plans all layers as one group."""
        n = ctypes.c_int32(0)
        ms = (ctypes.c_float * 36)()
        _check(self.lib.taot_get_group_trace(self.handle, ctypes.byref(n), ms), "taot_get_group_trace")
        return [[float(ms[g * 6 + i]) for i in range(6)] for g in range(n.value)]

    def match_cycles(self) -> torch.Tensor:
        """SM cycles per part of the matching + auction kernel of the last profiled call, int64 [L, 16] on the host
        (`taot_get_match_cycles`: set-up, Phase 2, Phase-3 set-up, Phase-3 bids, Phase-3 updates, whole kernel)."""
        out = torch.zeros((self.L, 16), dtype=torch.int64)
        _check(self.lib.taot_get_match_cycles(self.handle, _ptr(self.ws), _ptr(out)), "taot_get_match_cycles")
        return out

    # ------------------------------------------------------------------ stages
    def histogram(self, topk: torch.Tensor, info: Optional[torch.Tensor] = None):
        _dev(topk, torch.int32, "topk")
        L, R, E = self.L, self.R, self.E
        n = self._empty((L, R, E), torch.int32)
        el = self._empty((L, E), torch.int32)
        rl = self._empty((L, R), torch.int32)
        info = torch.zeros((L,), dtype=torch.int32, device=self.device) if info is None else info
        _check(self.lib.taot_histogram(self.handle, _ptr(topk), _ptr(n), _ptr(el), _ptr(rl), _ptr(info),
                                       _ptr(self.ws), _stream()), "taot_histogram")
        return n, el, rl, info

    def excess_spare(self, rank_load: torch.Tensor):
        _dev(rank_load, torch.int32, "rank_load")
        Bn, R = rank_load.shape
        ex = self._empty((Bn, R), torch.int32); sp = self._empty((Bn, R), torch.int32)
        s = self._empty((Bn, R), torch.float32); d = self._empty((Bn, R), torch.float32)
        _check(self.lib.taot_excess_spare(self.handle, _ptr(rank_load), ctypes.c_int32(Bn), _ptr(ex), _ptr(sp),
                                          _ptr(s), _ptr(d), _stream()), "taot_excess_spare")
        return ex, sp, s, d

    def sinkhorn(self, s: torch.Tensor, d: torch.Tensor, out: Optional[Dict[str, torch.Tensor]] = None):
        _dev(s, torch.float32, "s"); _dev(d, torch.float32, "d")
        Bn, R = s.shape
        if out is None:
            out = dict(plan=self._empty((Bn, R, R), torch.float32), iters=self._empty((Bn,), torch.int32),
                       row_err=self._empty((Bn,), torch.float32),
                       info=torch.zeros((Bn,), dtype=torch.int32, device=self.device))
        _check(self.lib.taot_sinkhorn(self.handle, _ptr(s), _ptr(d), ctypes.c_int32(Bn), _ptr(out["plan"]),
                                      _ptr(out["iters"]), _ptr(out["row_err"]), _ptr(out["info"]), _ptr(self.ws),
                                      _stream()), "taot_sinkhorn")
        return out

    def match(self, n, expert_load, rank_load, plan, info: Optional[torch.Tensor] = None):
        L, R, K, S = self.L, self.R, self.K, self.S
        se = self._empty((L, R, K), torch.int32); stk = self._empty((L, R, K), torch.int32)
        X = self._empty((L, R, S), torch.int32); rounds = self._empty((L, 2), torch.int32)
        info = torch.zeros((L,), dtype=torch.int32, device=self.device) if info is None else info
        _check(self.lib.taot_match(self.handle, _ptr(_dev(n, torch.int32, "n")),
                                   _ptr(_dev(expert_load, torch.int32, "expert_load")),
                                   _ptr(_dev(rank_load, torch.int32, "rank_load")),
                                   _ptr(None if plan is None else _dev(plan, torch.float32, "plan")), _ptr(se),
                                   _ptr(stk), _ptr(X),
                                   _ptr(rounds), _ptr(info), _ptr(self.ws), _stream()), "taot_match")
        return dict(slot_expert=se, slot_tokens=stk, X=X, rounds=rounds, info=info)

    def assign(self, topk, slot_expert, X, reuse_counts: bool = False, info: Optional[torch.Tensor] = None,
               out: Optional[torch.Tensor] = None):
        _dev(topk, torch.int32, "topk")
        new = torch.empty_like(topk) if out is None else out
        info = torch.zeros((self.L,), dtype=torch.int32, device=self.device) if info is None else info
        _check(self.lib.taot_assign(self.handle, _ptr(topk), _ptr(_dev(slot_expert, torch.int32, "slot_expert")),
                                    _ptr(_dev(X, torch.int32, "X")), _ptr(new), _ptr(info), _ptr(self.ws),
                                    ctypes.c_int32(1 if reuse_counts else 0), _stream()), "taot_assign")
        return new, info

    def dispatch(self, new_idx: torch.Tensor, info: Optional[torch.Tensor] = None, want_target_counts: bool = True,
                 out: Optional[Dict[str, torch.Tensor]] = None):
        """Send counts [L,R,R], target counts [L,R,E+S] and send-buffer positions [L,T,k] of a rewritten routing
        table, through `taot_dispatch`.  `out`: a dict returned by an earlier call, to reuse its tensors."""
        _dev(new_idx, torch.int32, "new_idx")
        L, R, E, S = self.L, self.R, self.E, self.S
        if out is not None:
            send, tc, perm, info = out["send_counts"], out["target_counts"], out["perm"], out["info"]
            info.zero_()
        else:
            send = self._empty((L, R, R), torch.int32)
            tc = self._empty((L, R, E + S), torch.int32) if want_target_counts else None
            perm = torch.empty_like(new_idx)
            info = torch.zeros((L,), dtype=torch.int32, device=self.device) if info is None else info
        _check(self.lib.taot_dispatch(self.handle, _ptr(new_idx), _ptr(send), _ptr(tc), _ptr(perm), _ptr(info),
                                      _ptr(self.ws), _stream()), "taot_dispatch")
        return dict(send_counts=send, target_counts=tc, perm=perm, info=info)

    def report(self, expert_load, rank_load, slot_expert, X, lam: float = 3.0) -> Dict[str, object]:
        """Dispatch diagnostics of L finished plans through `taot_report`.  Returns the row fields as numpy
        arrays of length L (named as in `ReportRow`) plus the tensors spill [L,E], load_after [L,R],
        slot_moved [L,S], slot_kind [L,S] (still on the device)."""
        import numpy as np
        L, R, E, S = self.L, self.R, self.E, self.S
        rows = torch.zeros((L, ctypes.sizeof(ReportRow)), dtype=torch.uint8, device=self.device)
        spill = self._empty((L, E), torch.int32); after = self._empty((L, R), torch.int32)
        moved = self._empty((L, S), torch.int32); kind = self._empty((L, S), torch.int32)
        _check(self.lib.taot_report(self.handle, _ptr(_dev(expert_load, torch.int32, "expert_load")),
                                    _ptr(_dev(rank_load, torch.int32, "rank_load")),
                                    _ptr(_dev(slot_expert, torch.int32, "slot_expert")),
                                    _ptr(_dev(X, torch.int32, "X")), ctypes.c_double(lam), _ptr(rows), _ptr(spill),
                                    _ptr(after), _ptr(moved), _ptr(kind), _stream()), "taot_report")
        raw = rows.cpu().numpy().tobytes()
        recs = (ReportRow * L).from_buffer_copy(raw)
        out: Dict[str, object] = {name: np.array([getattr(r, name) for r in recs]) for name, _ in ReportRow._fields_}
        out.update(spill=spill, load_after=after, slot_moved=moved, slot_kind=kind)
        return out

    # ------------------------------------------------------------------ whole path
    def _outputs_struct(self, out: Dict[str, torch.Tensor]) -> _Outputs:
        o = _Outputs()
        for name, _ in _Outputs._fields_:
            t = out.get(name)
            setattr(o, name, None if t is None else t.data_ptr())
        return o

    def plan(self, topk: torch.Tensor, out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        _dev(topk, torch.int32, "topk")
        out = self.alloc_outputs() if out is None else out
        o = self._outputs_struct(out)
        _check(self.lib.taot_plan(self.handle, _ptr(topk), ctypes.byref(o), _ptr(self.ws), _stream()), "taot_plan")
        return out

    def alloc_host_outputs(self, names=("plan", "slot_expert", "slot_tokens", "X", "new_idx", "info")):
        L, R, E, K, S, T, k = self.L, self.R, self.E, self.K, self.S, self.T, self.k
        shapes = dict(n=((L, R, E), torch.int32), expert_load=((L, E), torch.int32), rank_load=((L, R), torch.int32),
                      excess=((L, R), torch.int32), spare=((L, R), torch.int32), plan=((L, R, R), torch.float32),
                      sinkhorn_iters=((L,), torch.int32), row_err=((L,), torch.float32),
                      slot_expert=((L, R, K), torch.int32), slot_tokens=((L, R, K), torch.int32),
                      X=((L, R, S), torch.int32), rounds=((L, 2), torch.int32), new_idx=((L, T, k), torch.int32),
                      info=((L,), torch.int32))
        return {nm: torch.empty(shapes[nm][0], dtype=shapes[nm][1]).pin_memory() for nm in names}

    def alloc_host_block(self) -> Dict[str, torch.Tensor]:
        """Pinned host buffers for `plan_host_block`: the rewritten routing table, one block for every other output,
        and a view into the block per output (all 14 names of the outputs, plus "_block")."""
        offs = (ctypes.c_size_t * 14)()
        nbytes = ctypes.c_size_t()
        _check(self.lib.taot_host_block_layout(self.handle, offs, ctypes.byref(nbytes)), "taot_host_block_layout")
        L, R, E, K, S, T, k = self.L, self.R, self.E, self.K, self.S, self.T, self.k
        shapes = dict(n=((L, R, E), torch.int32), expert_load=((L, E), torch.int32), rank_load=((L, R), torch.int32),
                      excess=((L, R), torch.int32), spare=((L, R), torch.int32), plan=((L, R, R), torch.float32),
                      sinkhorn_iters=((L,), torch.int32), row_err=((L,), torch.float32),
                      slot_expert=((L, R, K), torch.int32), slot_tokens=((L, R, K), torch.int32),
                      X=((L, R, S), torch.int32), rounds=((L, 2), torch.int32), info=((L,), torch.int32))
        block = torch.empty(nbytes.value, dtype=torch.uint8).pin_memory()
        out = {"_block": block, "new_idx": torch.empty((L, T, k), dtype=torch.int32).pin_memory()}
        for i, (name, _) in enumerate(_Outputs._fields_):
            if name == "new_idx":
                continue
            shape, dt = shapes[name]
            count = 1
            for d in shape:
                count *= d
            out[name] = block[offs[i]: offs[i] + 4 * count].view(dt).view(shape)
        return out

    def plan_host_block(self, topk_host: torch.Tensor, out_host: Dict[str, torch.Tensor]) -> Dict[str, torch.Tensor]:
        """`plan_host` into buffers from `alloc_host_block`: two device-to-host copies for all outputs."""
        if topk_host.is_cuda or topk_host.dtype != torch.int32 or not topk_host.is_contiguous():
            raise TaotError("topk_host: expected a contiguous CPU int32 tensor")
        if "_block" not in out_host:
            raise TaotError("out_host: expected the buffers of alloc_host_block")
        if self._host_ws is None:
            self._host_ws = torch.empty(self.host_ws_bytes, dtype=torch.uint8, device=self.device)
        _check(self.lib.taot_plan_host_block(self.handle, _ptr(topk_host), _ptr(out_host["new_idx"]),
                                             _ptr(out_host["_block"]), _ptr(self._host_ws), _stream()),
               "taot_plan_host_block")
        return out_host

    def plan_host(self, topk_host: torch.Tensor, out_host: Dict[str, torch.Tensor]) -> Dict[str, torch.Tensor]:
        """Whole path from a HOST routing table to HOST results; copies ride the current stream."""
        if topk_host.is_cuda or topk_host.dtype != torch.int32 or not topk_host.is_contiguous():
            raise TaotError("topk_host: expected a contiguous CPU int32 tensor")
        if self._host_ws is None:
            self._host_ws = torch.empty(self.host_ws_bytes, dtype=torch.uint8, device=self.device)
        o = self._outputs_struct(out_host)
        _check(self.lib.taot_plan_host(self.handle, _ptr(topk_host), ctypes.byref(o), _ptr(self._host_ws),
                                       _stream()), "taot_plan_host")
        return out_host


def split_layers(L: int, groups: int):
    """Contiguous, near-equal split of L layers into at most `groups` non-empty groups: [(lo, hi), ...]."""
    groups = max(1, min(groups, L))
    base, extra = divmod(L, groups)
    bounds, lo = [], 0
    for g in range(groups):
        hi = lo + base + (1 if g < extra else 0)
        bounds.append((lo, hi))
        lo = hi
    return bounds


class PipelinedHostPlanner:
    """`taot_plan_host` over groups of layers on separate streams, so that the host-to-device copy of one group,
    the kernels of another and the device-to-host copy of a third overlap (the L problems of a call are
    independent, so splitting the batch changes no result).  Holds one `Planner` (handle, workspace, staging) per
    group; `plan_host` enqueues every group and makes the caller's current stream wait for all of them."""

    def __init__(self, L: int, groups: int = 4, **planner_kwargs):
        self.bounds = split_layers(L, groups)
        self.planners = [Planner(L=hi - lo, **planner_kwargs) for lo, hi in self.bounds]
        self.streams = [torch.cuda.Stream() for _ in self.planners]
        self.L = L
        self._key, self._calls, self._held = None, [], None

    def alloc_host_block(self) -> Dict[str, torch.Tensor]:
        """Packed host outputs (see `Planner.alloc_host_block`); only with a single group of layers."""
        if len(self.planners) != 1:
            raise TaotError("packed host outputs need a single group of layers")
        return self.planners[0].alloc_host_block()

    def alloc_host_outputs(self, names=("plan", "slot_expert", "slot_tokens", "X", "new_idx", "info")):
        parts = [p.alloc_host_outputs(names) for p in self.planners]
        # one pinned tensor per output, of which every group sees its slice
        out = {}
        for nm in names:
            shape = (self.L,) + tuple(parts[0][nm].shape[1:])
            out[nm] = torch.empty(shape, dtype=parts[0][nm].dtype).pin_memory()
        return out

    def plan_host(self, topk_host: torch.Tensor, out_host: Dict[str, torch.Tensor], join: bool = True) -> Dict[str, torch.Tensor]:
        if topk_host.is_cuda or topk_host.dtype != torch.int32 or not topk_host.is_contiguous():
            raise TaotError("topk_host: expected a contiguous CPU int32 tensor")
        if "_block" in out_host:                      # packed outputs: a single group, one call
            if len(self.planners) != 1:
                raise TaotError("packed host outputs need a single group of layers")
            cur = torch.cuda.current_stream()
            st = self.streams[0]
            st.wait_stream(cur)
            with torch.cuda.stream(st):
                self.planners[0].plan_host_block(topk_host, out_host)
            self._held = (topk_host, out_host)
            if join:
                self.join()
            return out_host
        # the per-group argument blocks depend only on the buffers' addresses: marshal them once per buffer set
        key = (topk_host.data_ptr(),) + tuple((k, v.data_ptr()) for k, v in sorted(out_host.items()))
        if key != self._key:
            calls = []
            for (lo, hi), pl in zip(self.bounds, self.planners):
                if pl._host_ws is None:
                    pl._host_ws = torch.empty(pl.host_ws_bytes, dtype=torch.uint8, device=pl.device)
                o = pl._outputs_struct({k: v[lo:hi] for k, v in out_host.items()})
                calls.append((pl, _ptr(topk_host[lo:hi]), o, _ptr(pl._host_ws)))
            self._calls, self._key, self._held = calls, key, (topk_host, out_host)
        cur = torch.cuda.current_stream()
        fn = self.planners[0].lib.taot_plan_host
        for (pl, tp, o, ws), st in zip(self._calls, self.streams):
            st.wait_stream(cur)
            _check(fn(pl.handle, tp, ctypes.byref(o), ws, ctypes.c_void_p(st.cuda_stream)), "taot_plan_host")
        if join:
            self.join()
        return out_host

    def join(self):
        """Make the caller's current stream wait for everything enqueued on the group streams."""
        cur = torch.cuda.current_stream()
        for st in self.streams:
            cur.wait_stream(st)

    def launch_count(self) -> int:
        return sum(p.last_launch_count() for p in self.planners)

    def plan_launches(self) -> int:
        return sum(p.plan_launches() for p in self.planners)

    def close(self):
        for p in self.planners:
            p.close()


class StreamingHostPlanner:
    """Several `taot_plan_host` calls in flight: `depth` pipelined planners (each with its own handles, workspaces,
    staging buffers and streams) take the submitted steps in turn, so that the copies of one step overlap the
    kernels of the previous one.  `submit` only enqueues; `result` blocks the host until that step's outputs are in
    host memory.  A lane is reused only after its previous step has finished (the submitting stream waits for it),
    so a caller must read a step's outputs before it submits `depth` further steps into the same output buffers."""

    def __init__(self, L: int, depth: int = 2, groups: int = 4, **planner_kwargs):
        if depth < 1:
            raise TaotError("depth must be at least 1")
        self.lanes = [PipelinedHostPlanner(L=L, groups=groups, **planner_kwargs) for _ in range(depth)]
        self.depth = depth
        self.L = L
        self._done = [torch.cuda.Event() for _ in range(depth)]
        self._busy = [False] * depth
        self._outs = [None] * depth
        self._n = 0

    def alloc_host_outputs(self, names=("plan", "slot_expert", "slot_tokens", "X", "new_idx", "info"), packed=None):
        """One pinned output set per lane.  packed (default: whenever a call is one group of layers): every output
        but the routing table lives in one block per lane and comes back in one copy (all outputs are then
        present, whatever `names` says)."""
        if packed is None:
            packed = all(len(lane.planners) == 1 for lane in self.lanes)
        if packed:
            return [lane.alloc_host_block() for lane in self.lanes]
        return [lane.alloc_host_outputs(names) for lane in self.lanes]

    def submit(self, topk_host: torch.Tensor, out_host: Dict[str, torch.Tensor]) -> int:
        """Enqueue one step; returns its ticket.  The current stream first waits for the lane's previous step."""
        lane = self._n % self.depth
        cur = torch.cuda.current_stream()
        if self._busy[lane]:
            cur.wait_event(self._done[lane])
        pl = self.lanes[lane]
        pl.plan_host(topk_host, out_host, join=False)
        # the lane's completion: an event on its first stream after that stream has waited for the others
        first = pl.streams[0]
        for st in pl.streams[1:]:
            first.wait_stream(st)
        self._done[lane].record(first)
        self._busy[lane] = True
        self._outs[lane] = out_host
        self._n += 1
        return self._n - 1

    def lane_of(self, ticket: int) -> int:
        return ticket % self.depth

    def wait_lane(self, lane: int):
        """Make the current stream wait for the step last submitted to this lane."""
        if self._busy[lane]:
            torch.cuda.current_stream().wait_event(self._done[lane])

    def result(self, ticket: int) -> Dict[str, torch.Tensor]:
        """Block the host until the step is complete; its outputs (valid until the lane's next submit)."""
        if ticket < self._n - self.depth or ticket >= self._n:
            raise TaotError("ticket is not in flight")
        lane = ticket % self.depth
        self._done[lane].synchronize()
        return self._outs[lane]

    def join(self):
        """Make the current stream wait for every step in flight."""
        for lane in range(self.depth):
            self.wait_lane(lane)

    def launch_count(self) -> int:
        return sum(l.launch_count() for l in self.lanes)

    def close(self):
        for l in self.lanes:
            l.close()
