#!/usr/bin/env python
"""Benchmark of the TAOT planner hot path on B200.

One step = one pass of the whole path (histogram -> excess/spare -> Sinkhorn -> matching +
auction -> token reassignment) over one batch of L synthetic routing problems, through
`taot_plan`.  Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl ours|reference]

The default workload is the largest single-GPU configuration (config 4: 48 layers, 256 ranks, a
1.6 GB routing table).  N > 1: one process per GPU.  Started under torch.distributed.run the ranks
come from the environment; started as a plain `python bench.py --gpus N` the script launches the N
ranks itself (torch.distributed.run, rendezvous on 127.0.0.1).  Every rank plans its own L problems
(independent replicas, no data-path collective), the timed region is bracketed by barriers and the
slowest rank's device time is reported.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
FLUSH_BYTES = 256 * 1024 * 1024
FP32_LANES_PER_SM = 128
# DRAM bytes per algorithmic byte of the streaming kernels, from one ncu capture each (config 3 shape with
# 8 layers; traffic grows in proportion to the entries processed, so a full launch is scaled by its own
# algorithmic bytes).  The reassignment figure is read + write once dirty L2 lines drain.
HIST_TRAFFIC_RATIO = 1.045
HIST_TRAFFIC_RATIO_BYTES = 1.01      # with the one-byte copy of the table written beside the counts (config 4 shape, 8 layers)
ASSIGN_TRAFFIC_RATIO = 1.01


def byte_table(cfg) -> bool:
    """The library's rule for leaving the routing table as one byte per entry in the histogram pass (which the
    reassignment then reads instead of the table): at most 256 experts, rank segments of a multiple of 16 entries."""
    return cfg.R <= 256 and cfg.E <= 256 and (cfg.T // cfg.R * cfg.k) % 16 == 0


def stream_bytes(cfg):
    """Algorithmic HBM bytes of the histogram and of the reassignment for one call: 4 B per entry read and 4 B per entry
    written in any case; with the byte table the histogram also writes 1 B per entry and the reassignment reads that byte
    instead of the entry (10 B per entry for the two kernels together instead of 12)."""
    entries = cfg.L * cfg.T * cfg.k
    if byte_table(cfg):
        return 5 * entries, 5 * entries
    return 4 * entries, 8 * entries
# the matching kernel reads its layer's counts, plan and lists once and keeps every round in shared memory: DRAM bytes per
# layer from one ncu capture at the config-4 shape (606 KB read, nothing written back by the end, for 2 layers)
MATCH_DRAM_BYTES_PER_LAYER = 303_000
STAGES = ["histogram", "merge", "sinkhorn", "match_auction", "assign"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="cfg4", choices=sorted(W.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="override L (smaller batch, e.g. for a profiler capture)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-groups", type=int, default=4,
                    help="layer groups (streams) the end-to-end host call is pipelined over")
    ap.add_argument("--e2e-depth", type=int, default=0,
                    help="host calls in flight in the end-to-end measurement (0: 4 for tables up to 64 MB, else 2)")
    ap.add_argument("--rendezvous-only", action="store_true",
                    help="check the launch path only: every rank joins the process group (gloo when there is no "
                         "GPU), the ranks reduce a per-rank time to the slowest one, rank 0 prints one JSON line")
    ap.add_argument("--e2e-stream-groups", type=int, default=1,
                    help="layer groups per call when several calls are in flight")
    ap.add_argument("--no-streams", action="store_true", help="skip the HBM-sized streaming report")
    ap.add_argument("--sweep", action="store_true",
                    help="config 5: time taot_sinkhorn alone over the (B, R, eps) grid and print one JSON object")
    ap.add_argument("--sweep-batches", type=int, nargs="+", default=[1, 64, 1024, 4096], help="batch sizes of --sweep")
    ap.add_argument("--sweep-ranks", type=int, nargs="+", default=[8, 16, 64, 256, 1024], help="rank counts of --sweep")
    ap.add_argument("--sweep-eps", type=float, nargs="+", default=[0.1, 0.01], help="eps / max(C) values of --sweep")
    ap.add_argument("--sweep-general-cost", action="store_true",
                    help="--sweep with a cost that has no tier structure (a tenth of the entries raised by 0.25): the "
                         "kernels that hold the kernel matrix, the clusters and the tensor-core products instead of the "
                         "tier-by-tier sums")
    ap.add_argument("--sweep-max-elems", type=float, default=6e9,
                    help="skip sweep cells whose plan tensor would exceed this many floats")
    return ap.parse_args()


# ---------------------------------------------------------------------------------------------
# clocks


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# ---------------------------------------------------------------------------------------------
# helpers


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), sm_max_mhz=float(d.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, sm_max_mhz=1965.0, source="fallback")


METRIC = "placement plans/s (whole planner path: histogram, excess/spare, Sinkhorn, matching+auction, token remap)"


def config_dict(args, cfg):
    """The `config` object of the JSON line; both arms print the same one for the same arguments."""
    table = cfg.L * cfg.T * cfg.k * 4
    return dict(workload=args.workload, L=cfg.L, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T,
                eps=cfg.eps, max_iters=cfg.max_iters, tol=cfg.tol, routing_table_bytes=table,
                l2="inputs larger than L2" if 2 * table >= 4 * L2_BYTES else "flushed between steps (256 MiB write)",
                parallelism=f"{max(1, args.gpus)} independent replica(s)")


def build_planner(cfg):
    import paper_2608_03676_b200 as P
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode)
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group)
    return P.Planner(L=cfg.L, R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r, C=C, eps=cfg.eps,
                     max_iters=cfg.max_iters, tol=cfg.tol)


def timed_steps(fn, steps, flush):
    """Device time of `steps` calls of fn, each bracketed by its own event pair; L2 flushed before each."""
    pairs = []
    for _ in range(steps):
        if flush is not None:
            flush.zero_()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record()
        pairs.append((a, b))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in pairs]


def oracle_sample(cfg, topk_cpu, seconds, threads=1):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: whole layers, taken round-robin
    (the workload is repeated if it is shorter than the budget) for about `seconds`.  threads > 1: that many
    layers at a time, one per host thread (the C routines release the interpreter lock)."""
    import oracle as O
    e2r = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode).numpy()
    C = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group).numpy()
    O.build()
    one = lambda l: O.plan_layers(topk_cpu[l:l + 1], cfg.R, cfg.E, cfg.K, e2r, C, cfg.eps, cfg.max_iters, cfg.tol)
    done, t_total = 0, 0.0
    if threads <= 1:
        while True:
            t0 = time.perf_counter()
            one(done % cfg.L)
            t_total += time.perf_counter() - t0
            done += 1
            if t_total + t_total / done > seconds:
                break
        return done, t_total
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=threads) as pool:
        while True:
            t0 = time.perf_counter()
            list(pool.map(one, [(done + i) % cfg.L for i in range(threads)]))
            t_total += time.perf_counter() - t0
            done += threads
            if t_total + t_total * threads / done > seconds:
                break
    return done, t_total


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def tiered_sums(C, B):
    """Does the library take the tier-by-tier Sinkhorn kernel for this cost matrix?  Its rule, applied to the matrix
    itself: 256, 512 or 1024 ranks and every off-diagonal cost equal to one of three values according to same node /
    same rail group / neither, with the block sizes read off the first row (ranks per node / per group 8 / 32, 4 / 16,
    4 / 32 or 16 / 32; a two-valued cost has no group tier)."""
    R = C.shape[0]
    if R not in (256, 512, 1024):
        return False
    row = C[0]
    node = 1
    while node < R and bool(row[node] == row[1]):
        node += 1
    group = node
    while group < R and bool(row[group] == row[min(node, R - 1)]):
        group += 1
    if group >= R:
        group = max(32, 2 * node)
    if (node, group) not in ((8, 32), (4, 16), (4, 32), (16, 32)) or R % group:
        return False
    i = torch.arange(R)
    same_node = (i[:, None] // node) == (i[None, :] // node)
    same_group = (i[:, None] // group) == (i[None, :] // group)
    want = torch.where(same_node, row[1], torch.where(same_group, row[node], row[min(group, R - 1)]))
    off = i[:, None] != i[None, :]
    return bool(torch.isfinite(want).all()) and bool((C[off] == want[off]).all())


def tiered_fma_per_iteration(R):
    """FMAs the tier-by-tier kernel executes per problem and iteration: per half-step one product per rank, the node
    and group factors, and three per rank for its own sum."""
    return 2 * (4 * R + R // 4 + 1)


def sinkhorn_chain_floor(out, cfg, lat):
    """Cycles of the dependent chain of ONE iteration of the kernel that solves this shape with few problems per
    call, from the measured latencies: shuffle-reduction levels, the two scaling updates, and the multiply-add
    chains in front of them.  None where no such model is kept (multi-warp tiles, clusters)."""
    ex = out["excess"].cpu().numpy(); sp = out["spare"].cpu().numpy()
    hn = int((ex > 0).sum(1).max()); cn = int((sp > 0).sum(1).max())
    if tiered_sums(W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group), cfg.L):
        # per half-step: node sum (two chains of four adds), node and group factors, five shuffle levels, three
        # multiply-adds of the rank's own sum, the scaling update
        return 2 * (5 * lat["shuffle_level"] + 9 * lat["fma"] + lat["rcp_mul"]), "2 x (5 shuffle levels + 9 fma + rcp-mul)"
    if cfg.R <= 64:
        # 4 x 8 lane grid: row sums over 8 column lanes (3 levels), column sums over 4 row lanes (2 levels); the
        # lane-local multiply-add chains are as long as the tile is deep (rows in steps of 4, columns in steps of 8)
        nra = max(1, -(-hn // 4)); ncg = max(2, -(-cn // 8))
        return (5 * lat["shuffle_level"] + (nra + ncg) * lat["fma"] + 2 * lat["rcp_mul"],
                f"5 shuffle levels + {nra + ncg} fma + 2 rcp-mul")
    return None, None


def sinkhorn_work(out, cfg):
    """FMA count the Sinkhorn kernel executed: 2 mat-vecs over the |hot| x |cold| block per iteration, or the
    tier-by-tier sums where the library takes those."""
    ex = out["excess"].cpu().numpy(); sp = out["spare"].cpu().numpy(); it = out["sinkhorn_iters"].cpu().numpy()
    hn = (ex > 0).sum(1).astype(np.int64); cn = (sp > 0).sum(1).astype(np.int64)
    if tiered_sums(W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group), cfg.L):
        return int((tiered_fma_per_iteration(cfg.R) * np.maximum(it - 1, 0)).sum()), it
    return int((2 * hn * cn * np.maximum(it - 1, 0)).sum()), it


def roofline_for(stage, ms, cfg, out, peaks, sm_count, match_cyc=None):
    topk_bytes = cfg.L * cfg.T * cfg.k * 4
    hbm = peaks["hbm_gbs"]
    hist_bytes, assign_bytes = stream_bytes(cfg)
    if stage == "histogram":
        a = hist_bytes / (ms * 1e-3) / 1e9
        return dict(kernel="hist_chunk_kernel", bound="hbm", achieved=a, peak=hbm, unit="GB/s", frac=a / hbm,
                    traffic=(HIST_TRAFFIC_RATIO_BYTES if byte_table(cfg) else HIST_TRAFFIC_RATIO) * hist_bytes,
                    peak_source=peaks["source"], bytes_per_launch=hist_bytes,
                    byte_table=byte_table(cfg))
    if stage == "assign":
        a = assign_bytes / (ms * 1e-3) / 1e9
        return dict(kernel="assign_chunk_kernel", bound="hbm", achieved=a, peak=hbm, unit="GB/s",
                    frac=a / hbm, traffic=ASSIGN_TRAFFIC_RATIO * assign_bytes, peak_source=peaks["source"],
                    bytes_per_launch=assign_bytes, byte_table=byte_table(cfg))
    if stage == "merge":
        b = cfg.L * cfg.R * cfg.E * 4 * (2 + max(1, (cfg.T // cfg.R * cfg.k + 16383) // 16384))
        a = b / (ms * 1e-3) / 1e9
        return dict(kernel="merge_kernel", bound="hbm", achieved=a, peak=hbm, unit="GB/s", frac=a / hbm,
                    traffic=None, peak_source=peaks["source"], bytes_per_launch=b,
                    note="one CTA per layer over a few tens of MB of chunk counts: a short kernel in the chain of "
                         "latency-bound stages, far from any bandwidth bound by construction")
    derived = sm_count * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    fp32_peak = peaks.get("fma_tflops") or derived
    fp32_src = (f"measured: taot_measure_alu_peaks (FMA chain kernel; ex2 {peaks.get('ex2_tops', 0):.2f} T/s); "
                f"derived figure {derived:.1f}") if peaks.get("fma_tflops") else \
        f"derived: {sm_count} SMs x 128 fp32 lanes x 2 x {peaks['sm_max_mhz']:.0f} MHz"
    if stage == "sinkhorn":
        fma, _ = sinkhorn_work(out, cfg)
        a = 2 * fma / (ms * 1e-3) / 1e12
        tiered = tiered_sums(W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group), cfg.L)
        latency = None
        if peaks.get("latency_cycles"):
            cyc, model = sinkhorn_chain_floor(out, cfg, peaks["latency_cycles"])
            if cyc:
                its = int(out["sinkhorn_iters"].max().item())
                floor_ns = cyc / (peaks["sm_max_mhz"] * 1e-3)
                ach_ns = ms * 1e6 / max(its, 1)
                latency = dict(bound="dependent chain of one iteration", floor_ns_per_iteration=floor_ns,
                               achieved_ns_per_iteration=ach_ns, frac=floor_ns / ach_ns, iterations=its, model=model,
                               cycles=peaks["latency_cycles"],
                               note="achieved = stage time / iterations of the slowest problem (set-up and "
                                    "write-out included); floor from taot_measure_latencies at the maximum SM clock")
        d = dict(kernel="sinkhorn_tiered_mw_kernel" if tiered else "sinkhorn_tile_kernel", bound="alu", achieved=a,
                    peak=fp32_peak, unit="TFLOP/s",
                    frac=a / fp32_peak, traffic=None,
                    peak_source=fp32_src, flops_per_launch=2 * fma,
                    note="one dependent chain of small mat-vecs per problem and only L problems per call: "
                         "latency-bound; DRAM traffic is ~0.1 MB per launch (ncu); the fp32-FMA fraction is "
                         "reported, not claimed as the binding limit (`bench.py --sweep` times batches that fill "
                         "the GPU)")
        if latency:
            d["latency"] = latency
        return d
    rounds = out["rounds"].cpu().numpy().astype(np.int64)
    ops = int((rounds[:, 0] * cfg.R * cfg.E + rounds[:, 1] * cfg.R * cfg.S).sum())
    a = ops / (ms * 1e-3) / 1e12
    d = dict(kernel="match_kernel", bound="alu", achieved=a, peak=fp32_peak / 2, unit="Tscore/s",
             frac=a / (fp32_peak / 2), traffic=MATCH_DRAM_BYTES_PER_LAYER * cfg.L,
             peak_source="half the FP32 FMA peak: one fp32 score evaluation per lane per clock",
             note="dependent rounds of masked arg-max, one CTA per layer; the figure counts the dense scores of the "
                  "paper's formulation (rounds x R x E and rounds x R x S) and no bandwidth or FLOP bound applies: "
                  "the stage is as long as its slowest layer's chain of rounds, see `rounds`")
    if match_cyc is not None:
        # the layer that takes longest; cycles as thread 0 of its CTA counts them (the counting build of the kernel is
        # ~10 % slower than the timed one, so the split is given in cycles and as shares, not as a time)
        w = int(match_cyc[:, 5].argmax())
        c = match_cyc[w]
        r2, r3 = int(rounds[w, 0]), int(rounds[w, 1])
        d["rounds"] = dict(
            slowest_layer=w, phase2_rounds=r2, phase3_rounds=r3, kernel_cycles=c[5],
            share=dict(setup=(c[0] + c[2]) / c[5], phase2=c[1] / c[5], phase3_rounds=c[12] / c[5]),
            phase2_cycles_per_round=c[1] / max(1, r2),
            phase3_cycles_per_round=dict(whole_round=c[12] / max(1, r3), bid_to_first_barrier=c[3] / max(1, r3), update_to_second_barrier=c[4] / max(1, r3),
                                         busiest_thread_probe=c[6] / max(1, r3), busiest_thread_arbitration=c[7] / max(1, r3)),
            phase2_split=dict(scan_and_arbitration=c[8], winners=c[9], served_rows=c[10], all_keys_per_slot_index=c[11]),
            ns_per_phase3_round_at_max_clock=c[12] / max(1, r3) / (peaks["sm_max_mhz"] * 1e-3),
            note="cycle counts of the counting build of the kernel (every thread reads the clock three times a round): "
                 "an upper bound on the timed build, whose stage time is `stages_ms.match_auction`; a barrier holds a "
                 "warp up at its next shared-memory access, so the wait at the first barrier of a round (for the warps "
                 "whose cursors move) is counted under update_to_second_barrier and the wait at the second under "
                 "bid_to_first_barrier of the next round")
        rl = peaks.get("round_latency_cycles")
        if rl and r3 > 0:
            # One auction round as a dependent chain: the probe (two independent shared-memory loads, AND, find-first-set,
            # rank index), the arbitration (atomicMax, barrier, read-back: measured as a unit), the winner's update
            # (load of its holding, subtract, store) and the closing barrier; six dependent integer operations at the
            # latency of a multiply-add stand for the ALU steps in between.
            fma = (peaks.get("latency_cycles") or {}).get("fma", 4.0)
            floor_cyc = 2 * rl["shared_load"] + rl["arbitration"] + rl["barrier"] + 6 * fma
            share3 = c[12] / c[5]
            ach_ns = ms * 1e6 * share3 / r3
            floor_ns = floor_cyc / (peaks["sm_max_mhz"] * 1e-3)
            d["latency"] = dict(bound="dependent chain of one auction round", floor_ns_per_round=floor_ns,
                                achieved_ns_per_round=ach_ns, frac=floor_ns / ach_ns, rounds=r3, cycles=rl,
                                model="2 shared loads + (atomicMax, barrier, read-back) + barrier + 6 integer operations",
                                note="achieved = stage time x the Phase-3 share of the slowest layer's cycles / its "
                                     "rounds; floor from taot_measure_round_latencies (eight warps, one CTA per SM) at "
                                     "the maximum SM clock")
    return d


def rank_config(cfg, rank: int):
    """Every rank plans its own batch: same shape, seed offset by rank (independent replicas)."""
    return cfg.replace(seed=cfg.seed + 7919 * rank)


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's device time (the step time of a synchronous job)."""
    import torch.distributed as dist
    t = torch.tensor([float(ms)], device=device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step: int, steps: int, world: int, slowest_ms: float) -> float:
    return world * units_per_rank_per_step * steps / (slowest_ms * 1e-3)


def dispatch_timing(pl, out, table_bytes, peaks, steps, flush):
    """The step after the path: dispatch metadata of the rewritten table (12 B per entry: two reads of the table,
    one write of the positions).  Not part of the timed planner step."""
    dsp = pl.dispatch(out["new_idx"])
    timed_steps(lambda: pl.dispatch(out["new_idx"], out=dsp), 2, flush)
    ms = float(np.mean(timed_steps(lambda: pl.dispatch(out["new_idx"], out=dsp), steps, flush)))
    gbs = 3 * table_bytes / (ms * 1e-3) / 1e9
    return dict(dispatch_ms=ms, dispatch_gbs=gbs, dispatch_frac=gbs / peaks["hbm_gbs"])


def stream_report(name, peaks, steps=5, flush=None):
    """Per-stage times of another workload: GB/s of the histogram and the reassignment (an HBM figure where the
    routing table is larger than L2; otherwise L2 is flushed between steps and the entry says so)."""
    cfg = W.get_config(name)
    topk = W.routing_topk(cfg, device="cuda")
    pl = build_planner(cfg)
    out = pl.alloc_outputs()
    b = topk.numel() * 4
    if 2 * b >= 4 * L2_BYTES:
        flush = None
    for _ in range(3):
        pl.plan(topk, out)
    call_ms = float(np.mean(timed_steps(lambda: pl.plan(topk, out), steps, flush)))      # the call as a user makes it
    pl.set_profiling(True)
    acc = np.zeros(5)
    for _ in range(steps):
        if flush is not None:
            flush.zero_()
        pl.plan(topk, out)
        acc += np.array(pl.stage_ms())
    acc /= steps
    pl.set_profiling(False)
    rep = dict(workload=name, topk_bytes=b, table_larger_than_l2=2 * b >= 4 * L2_BYTES,
               stages_ms=dict(zip(STAGES, [float(x) for x in acc])), stages_sum_ms=float(acc.sum()), ms_per_step=call_ms,
               histogram_gbs=stream_bytes(cfg)[0] / (acc[0] * 1e-3) / 1e9, assign_gbs=stream_bytes(cfg)[1] / (acc[4] * 1e-3) / 1e9,
               byte_table=byte_table(cfg),
               peak_gbs=peaks["hbm_gbs"], peak_source=peaks["source"],
               remapped_tokens_per_s=cfg.L * cfg.T / (acc[4] * 1e-3),
               plans_per_s=cfg.L / (call_ms * 1e-3))
    rep["histogram_frac"] = rep["histogram_gbs"] / peaks["hbm_gbs"]
    rep["assign_frac"] = rep["assign_gbs"] / peaks["hbm_gbs"]
    rep.update(dispatch_timing(pl, out, b, peaks, steps, flush))
    pl.close()
    del topk, out
    torch.cuda.empty_cache()
    return rep


# ---------------------------------------------------------------------------------------------
# arms


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = W.get_config(args.workload)
    if args.layers > 0:
        cfg = cfg.replace(L=args.layers)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    per_step = max(2.0, min(args.cpu_seconds, 60.0 / max(1, args.steps + args.warmup)))
    # the sample never needs more layers than steps x (layers one step gets through); a quarter of the workload
    # bounds the input generation when there is no GPU to draw it on
    n_gen = cfg.L if dev == "cuda" else max(1, min(cfg.L, 12, args.steps + args.warmup))
    topk = W.routing_topk(cfg, device=dev, layers=range(n_gen)).cpu().numpy()
    full = cfg
    cfg = cfg.replace(L=n_gen)
    layers, secs = 0, 0.0
    for i in range(args.warmup + args.steps):
        n, t = oracle_sample(cfg, topk, per_step)
        if i >= args.warmup:
            layers += n; secs += t
    value = layers / secs
    line = dict(metric=METRIC, value=value, unit="plans/s", n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * secs / max(1, args.steps),
                layers_per_step=layers / max(1, args.steps),
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                impl="reference", config=config_dict(args, full),
                cpu_baseline=dict(value=value, unit="plans/s", cores=1, kind="oracle",
                                  sample=f"{layers / max(1, args.steps):.1f} whole layer(s) per step of the "
                                         f"{full.L}-layer workload (taken round-robin from its first {n_gen})",
                                  cpu=cpu_model()),
                e2e=dict(value=value, unit="plans/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def run_ours(args):
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the planner has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()

    cfg = W.get_config(args.workload)
    if args.layers > 0:
        cfg = cfg.replace(L=args.layers)
    cfg = rank_config(cfg, rank)
    peaks = measured_peaks()
    import paper_2608_03676_b200 as P
    peaks.update(P.measure_alu_peaks())              # FP32-FMA and ex2 ceilings of this GPU, measured once, untimed
    peaks["latency_cycles"] = P.measure_latencies() # dependent-operation latencies, for the chain floor of the Sinkhorn stage
    peaks["round_latency_cycles"] = P.measure_round_latencies()   # the operations an auction round is a chain of
    props = torch.cuda.get_device_properties(local)
    topk = W.routing_topk(cfg, device="cuda")
    pl = build_planner(cfg)
    out = pl.alloc_outputs()
    topk_bytes = topk.numel() * 4
    need_flush = 2 * topk_bytes < 4 * L2_BYTES
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda") if need_flush else None

    step = lambda: pl.plan(topk, out)
    timed_steps(step, max(3, args.warmup), flush)
    barrier(); torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms = timed_steps(step, args.steps, flush)
    torch.cuda.synchronize(); barrier()
    launches = pl.last_launch_count() * args.steps
    # per-kernel durations inside the same step, from events the library records between its kernels
    pl.set_profiling(True)
    stage_ms = np.zeros(5)
    for _ in range(args.steps):
        if flush is not None:
            flush.zero_()
        pl.plan(topk, out)
        stage_ms += np.array(pl.stage_ms())
    stage_ms /= args.steps
    clocks = sampler.stop() if rank == 0 else None
    # where the matching kernel's time goes (cycle counters inside the kernel, one untimed call) and the timeline of
    # the layer groups of an overlapped call (one untimed call with per-group events)
    pl.set_profiling(2)
    pl.plan(topk, out)
    match_cyc = pl.match_cycles().numpy().astype(np.float64)
    pl.set_profiling(3)
    pl.plan(topk, out)
    group_trace = pl.group_trace()
    pl.set_profiling(False)
    dispatch = dispatch_timing(pl, out, topk_bytes, peaks, args.steps, flush) if world == 1 else None

    total_s = max_over_ranks(sum(ms), world, "cuda") * 1e-3
    value = whole_job_rate(cfg.L, args.steps, world, total_s * 1e3)

    # the same step replayed from a CUDA graph (captured once, untimed): launch gaps shrink, the kernels are the same
    graph_ms = None
    if world == 1:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            pl.plan(topk, out)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            pl.plan(topk, out)
        timed_steps(g.replay, 3, flush)
        graph_ms = timed_steps(g.replay, args.steps, flush)

    # end to end through the host-buffer entry point
    host_in = topk.cpu().pin_memory()
    e2r_h = W.expert_to_rank(cfg.E, cfg.R, cfg.e2r_mode)
    C_h = W.cost_matrix(cfg.R, cfg.gpus_per_node, cfg.tiers, cfg.nodes_per_group)
    depth = args.e2e_depth if args.e2e_depth > 0 else (4 if topk_bytes <= (64 << 20) else 2)
    kw = dict(R=cfg.R, E=cfg.E, K=cfg.K, k=cfg.k, T=cfg.T, e2r=e2r_h, C=C_h, eps=cfg.eps, max_iters=cfg.max_iters,
              tol=cfg.tol)
    names = ("plan", "slot_expert", "slot_tokens", "X", "new_idx", "info")
    # what the host link allows: one pinned copy of the routing table each way (the two directions of a step can
    # overlap, so the slower direction bounds a step that moves the table in and the rewritten table out)
    dev_buf = torch.empty_like(topk)
    back = torch.empty_like(host_in).pin_memory()
    link = {}
    for nm, fn in (("h2d", lambda: dev_buf.copy_(host_in, non_blocking=True)),
                   ("d2h", lambda: back.copy_(dev_buf, non_blocking=True))):
        fn(); torch.cuda.synchronize()
        link[nm] = topk_bytes / (min(timed_steps(fn, 3, None)) * 1e-3) / 1e9
    # both directions at once (what a stream of steps asks of the link: the table of step i+1 in while that of step i
    # goes out): two streams, one copy each way, timed from the first to the last
    dev_buf2 = torch.empty_like(topk)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    duplex = []
    for _ in range(3):
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True); e2 = torch.cuda.Event(enable_timing=True)
        e0.record()
        s1.wait_event(e0); s2.wait_event(e0)
        with torch.cuda.stream(s1):
            dev_buf.copy_(host_in, non_blocking=True); e1.record()
        with torch.cuda.stream(s2):
            back.copy_(dev_buf2, non_blocking=True); e2.record()
        torch.cuda.synchronize()
        duplex.append(max(e0.elapsed_time(e1), e0.elapsed_time(e2)))
    link["duplex_ms"] = float(min(duplex))
    del dev_buf, dev_buf2, back
    link_ms = topk_bytes / (min(link["h2d"], link["d2h"]) * 1e9) * 1e3
    # (a) one call at a time, pipelined over groups of layers inside the call: every step waits for the previous one
    hp = P.PipelinedHostPlanner(L=cfg.L, groups=args.e2e_groups, **kw)
    host_out = hp.alloc_host_outputs(names)
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())
    e2e_step = lambda: hp.plan_host(host_in, host_out)
    timed_steps(e2e_step, 3, flush)
    barrier(); torch.cuda.synchronize()
    serial_ms = timed_steps(e2e_step, args.steps, flush)
    serial_value = whole_job_rate(cfg.L, args.steps, world, max_over_ranks(sum(serial_ms), world, "cuda"))
    n_groups = len(hp.planners)
    hp.close(); del host_out
    sp = P.StreamingHostPlanner(L=cfg.L, depth=depth, groups=args.e2e_stream_groups, **kw)
    host_outs = sp.alloc_host_outputs(names)
    packed = "_block" in host_outs[0]
    if packed:                                       # one block (every output but the routing table) + the table
        d2h = host_outs[0]["_block"].numel() + host_outs[0]["new_idx"].numel() * 4

    # (b) `depth` calls in flight: step i starts once step i - depth has delivered its outputs (and L2 has been
    # flushed after that), while the steps between them are still copying and computing
    def streamed(steps):
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(steps):
            sp.wait_lane(i % depth)
            if flush is not None:
                flush.zero_()
            sp.submit(host_in, host_outs[i % depth])
        sp.join()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    streamed(3 * depth)
    barrier(); torch.cuda.synchronize()
    e2e_total_ms = streamed(args.steps)
    e2e_ms = [e2e_total_ms / args.steps]
    e2e_value = whole_job_rate(cfg.L, args.steps, world, max_over_ranks(e2e_total_ms, world, "cuda"))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    dominant = int(np.argmax(stage_ms))
    roof = roofline_for(STAGES[dominant], float(stage_ms[dominant]), cfg, out, peaks, props.multi_processor_count, match_cyc)
    fma, iters = sinkhorn_work(out, cfg)
    rounds = out["rounds"].cpu().numpy()
    info = out["info"].cpu().numpy()
    line = dict(
        metric=METRIC,
        value=value, unit="plans/s", n_gpus=world, steps=args.steps, warmup=max(3, args.warmup),
        ms_per_step=float(np.mean(ms)), ms_per_step_median=float(np.median(ms)), ms_per_step_min=float(np.min(ms)),
        higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f32",
        data="synthetic",
        config=config_dict(args, cfg),
        remapped_tokens_per_s=cfg.L * cfg.T / (float(stage_ms[4]) * 1e-3),
        histogram_tokens_per_s=cfg.L * cfg.T / (float(stage_ms[0]) * 1e-3),
        planned_tokens_per_s=world * cfg.L * cfg.T * args.steps / total_s,
        stages_ms=dict(zip(STAGES, [float(x) for x in stage_ms])),
        sinkhorn=dict(iters_mean=float(iters.mean()), iters_max=int(iters.max()),
                      converged_frac=float(((info & 2) == 0).mean()),
                      plans_per_s=cfg.L / (float(stage_ms[2]) * 1e-3)),
        rounds=dict(phase2_max=int(rounds[:, 0].max()), phase3_max=int(rounds[:, 1].max())),
        roofline=roof, clocks=clocks,
        e2e=dict(value=e2e_value, unit="plans/s", h2d_bytes_per_step=topk_bytes, d2h_bytes_per_step=d2h,
                 ms_per_step=float(np.mean(e2e_ms)), in_flight=depth,
                 host_link=dict(h2d_gbs=link["h2d"], d2h_gbs=link["d2h"], bound_ms_per_step=link_ms,
                                bound_value=world * cfg.L / (link_ms * 1e-3),
                                both_directions_ms_per_step=link["duplex_ms"],
                                both_directions_value=world * cfg.L / (link["duplex_ms"] * 1e-3),
                                note="pinned copies of the routing table alone: each way by itself (the slower direction "
                                     "bounds a step that moves the table in and the rewritten table out), and both ways "
                                     "at once on two streams, which is what a stream of steps asks of the link"),
                 serial_value=serial_value, serial_ms_per_step=float(np.mean(serial_ms)),
                 api=f"StreamingHostPlanner.submit: {'taot_plan_host_block (outputs packed: two copies back)' if packed else 'taot_plan_host'}, {depth} call(s) in flight, each on "
                     f"{len(sp.lanes[0].planners)} group(s) of layers; serial_*: PipelinedHostPlanner.plan_host, one "
                     f"call at a time on {n_groups} groups of layers (one stream each)"),
        gpu_launches=launches,
    )
    if dispatch is not None:
        line["dispatch"] = dict(dispatch, note="taot_dispatch on the rewritten table, outside the timed step")
    if graph_ms is not None:
        line["cuda_graph"] = dict(ms_per_step=float(np.mean(graph_ms)), value=cfg.L / (float(np.mean(graph_ms)) * 1e-3),
                                  unit="plans/s", note="the same taot_plan call captured once and replayed")
    line["rooflines"] = {s: roofline_for(s, float(stage_ms[i]), cfg, out, peaks, props.multi_processor_count, match_cyc)
                         for i, s in enumerate(STAGES)}
    line["stages_note"] = ("stages_ms: the call planned as one group of layers on one stream (stage events); ms_per_step: "
                           "the call as a user makes it, which for a table this large overlaps layer groups on internal "
                           "streams, so it is shorter than the sum of the stages")
    if group_trace:
        line["layer_groups"] = dict(
            groups=len(group_trace), columns=["start", "histogram", "merge", "sinkhorn", "match_auction", "assign"],
            ms_from_call_start=group_trace,
            note="one untimed call with per-group events: when each group of layers finished each stage")

    if world == 1 and not args.no_streams:
        del host_in, host_outs
        sp.close()
        torch.cuda.empty_cache()
        fl = flush if flush is not None else torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
        line["hbm_streams"] = [stream_report(nm, peaks) for nm in ("cfg3", "cfg4") if nm != args.workload]
        line["l2_resident_workloads"] = [stream_report(nm, peaks, flush=fl) for nm in ("cfg2",) if nm != args.workload]
    if world == 1 and not args.no_cpu_baseline:
        n_layers, secs = oracle_sample(cfg, topk.cpu().numpy(), args.cpu_seconds)
        line["cpu_baseline"] = dict(value=n_layers / secs, unit="plans/s", cores=1, kind="oracle",
                                    sample=f"{n_layers} whole layer(s) (the {cfg.L}-layer workload taken round-robin), "
                                           f"{secs:.2f} s", cpu=cpu_model())
        cores = max(1, min(len(os.sched_getaffinity(0)), cfg.L))
        if cores > 1:
            n_mt, secs_mt = oracle_sample(cfg, topk.cpu().numpy(), max(2.0, args.cpu_seconds / 4), threads=cores)
            line["cpu_baseline_threads"] = dict(value=n_mt / secs_mt, unit="plans/s", cores=cores, kind="oracle",
                                                sample=f"{n_mt} whole layer(s), one per host thread, {secs_mt:.2f} s")
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Config 5: Sinkhorn only.  Per cell: plans/s and the executed-FMA fraction of the fp32 peak."""
    import paper_2608_03676_b200 as P
    from workloads.configs import SWEEP_ITERS, SWEEP_TIERS
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    props = torch.cuda.get_device_properties(0)
    alu = P.measure_alu_peaks()
    fp32_peak = alu["fma_tflops"]                    # measured FMA-chain throughput of this GPU
    # dense TF32 ceiling: the measured bf16 GEMM burst figure times the nominal TF32 : bf16 ratio (1.1 : 2.25 PFLOP/s)
    try:
        bf16 = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
        tf32_src = "measured bf16 GEMM burst x nominal ratio 1.1 / 2.25"
    except Exception:
        bf16, tf32_src = 1590.0, "fallback bf16 figure x nominal ratio 1.1 / 2.25"
    tf32_peak = bf16 * 1.1 / 2.25
    cells = []
    cells_todo = W.sweep_cells(batches=tuple(args.sweep_batches), ranks=tuple(args.sweep_ranks),
                               eps_fracs=tuple(args.sweep_eps))
    for (B, R, eps_frac) in cells_todo:
        if B * R * R > args.sweep_max_elems:
            cells.append(dict(B=B, R=R, eps_frac=eps_frac, skipped="plan tensor larger than --sweep-max-elems"))
            continue
        C = W.cost_matrix(R, 8, SWEEP_TIERS, 4)
        if args.sweep_general_cost:
            ii = torch.arange(R)
            C = C + 0.25 * (((ii[:, None] * 5 + ii[None, :] * 3) % 11 == 0) & (ii[:, None] != ii[None, :])).to(C.dtype)
        pl = P.Planner(L=B, R=R, E=R, K=1, k=1, T=R, e2r=torch.arange(R, dtype=torch.int32), C=C,
                       eps=eps_frac * max(SWEEP_TIERS), max_iters=SWEEP_ITERS, tol=0.0)
        loads = W.sweep_rank_loads(B, R, seed=5000 + R, device="cuda")
        ex, sp, s, d = pl.excess_spare(loads)
        out = pl.sinkhorn(s, d)
        reps = 3 if B * R * R < 5e8 else 1
        ms = timed_steps(lambda: pl.sinkhorn(s, d, out), reps + 1, None)[1:]
        hn = (ex > 0).sum(1).double(); cn = (sp > 0).sum(1).double()
        dense_fma = float((2 * hn * cn * (SWEEP_ITERS - 1)).sum())        # a solver that holds the kernel matrix
        tiered = tiered_sums(C, B)
        fma = float(B * tiered_fma_per_iteration(R) * (SWEEP_ITERS - 1)) if tiered else dense_fma
        t = float(np.median(ms)) * 1e-3
        # the library's rule for the dense products on the tensor cores, mirrored
        tensor = (not tiered and R > 256 and R % 128 == 0 and B >= 256 and float(C.max()) / (eps_frac * max(SWEEP_TIERS)) <= 20.0
                  and not os.environ.get("TAOT_NO_TENSOR_CORES"))
        if tensor:
            # executed: per iteration two products [R,R] x [R,B], each as three TF32 products
            tc_flops = 2.0 * 3.0 * 2.0 * R * R * B * SWEEP_ITERS
            cells.append(dict(B=B, R=R, eps_frac=eps_frac, ms=t * 1e3, plans_per_s=B / t, kernel="tensor-core products (3 x TF32)",
                              tflops=tc_flops / t / 1e12, frac_tf32_peak=tc_flops / t / 1e12 / tf32_peak,
                              tf32_peak_tflops=tf32_peak, useful_tflops=tc_flops / 3.0 / t / 1e12,
                              matrix_equiv_tflops=2 * dense_fma / t / 1e12,
                              hot_mean=float(hn.mean()), cold_mean=float(cn.mean()), info_or=int(out["info"].max())))
            pl.close()
            del out, loads, s, d, ex, sp
            torch.cuda.empty_cache()
            continue
        cells.append(dict(B=B, R=R, eps_frac=eps_frac, ms=t * 1e3, plans_per_s=B / t,
                          kernel="tiered sums" if tiered else "kernel matrix",
                          tflops=2 * fma / t / 1e12, frac_fp32_peak=2 * fma / t / 1e12 / fp32_peak,
                          matrix_equiv_tflops=2 * dense_fma / t / 1e12,
                          hot_mean=float(hn.mean()), cold_mean=float(cn.mean()),
                          info_or=int(out["info"].max())))
        pl.close()
        del out, loads, s, d, ex, sp
        torch.cuda.empty_cache()
    print(json.dumps(dict(metric="Sinkhorn placement plans/s per (B, R, eps) cell, 500 fixed iterations",
                          unit="plans/s", fp32_peak_tflops=fp32_peak, ex2_peak_tops=alu["ex2_tops"],
                          fp32_peak_source="measured: taot_measure_alu_peaks", tf32_peak_tflops=tf32_peak,
                          tf32_peak_source=tf32_src, general_cost=bool(args.sweep_general_cost),
                          fp32_peak_derived=props.multi_processor_count * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12,
                          cells=cells)))


def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def launch_ranks(args, argv) -> int:
    """`python bench.py --gpus N` outside a launcher: start the N ranks (one process per GPU) under
    torch.distributed.run on this node and hand back its exit code.  Rank 0's JSON line goes to this process's
    stdout unchanged."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    env = dict(os.environ)
    env.setdefault("OMP_NUM_THREADS", "1")
    return subprocess.call(cmd, env=env)


def run_rendezvous_only(args):
    """The launch path without the planner: join the process group (nccl on GPUs, gloo without), reduce a per-rank
    time to the slowest rank's as the timed arms do, and print what the ranks saw."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    gpu = torch.cuda.is_available()
    if gpu:
        torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl" if gpu else "gloo")
    dev = "cuda" if gpu else "cpu"
    cfg = rank_config(W.get_config(args.workload), rank)
    slowest = max_over_ranks(10.0 * (rank + 1), world, dev)
    seeds = [None] * world
    if world > 1:
        dist.all_gather_object(seeds, cfg.seed)
        dist.barrier()
    else:
        seeds = [cfg.seed]
    if rank == 0:
        print(json.dumps(dict(rendezvous_only=True, n_gpus=world, gpus_requested=args.gpus,
                              backend=("nccl" if gpu else "gloo") if world > 1 else None, slowest_ms=slowest,
                              seeds=seeds, value=whole_job_rate(cfg.L, 1, world, slowest), unit="plans/s")))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.sweep:
        raise SystemExit(launch_ranks(args, sys.argv[1:]))
    if args.rendezvous_only:
        run_rendezvous_only(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
