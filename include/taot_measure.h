/*
 * taot_measure.h -- measurement aids of libtaot: stage timing, cycle counters of the matching kernel, the timeline of
 * the layer groups, and the arithmetic ceilings / latencies of the device.  None of these is a step of the planner
 * (the paper has no counterpart for any of them) and nothing in taot.h depends on them; they are exported by the same
 * library for benchmarks and profiles.
 */
#ifndef TAOT_MEASURE_H
#define TAOT_MEASURE_H

#include "taot.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Stage timing for benchmarks.  With profiling on, taot_plan (and taot_plan_host) records one CUDA
 * event on `stream` before the first kernel and one after each of its five stages (chunk
 * histogram; merge; Sinkhorn; matching + auction; reassignment = table build + rewrite kernels).
 * taot_get_stage_ms waits for the last of them and returns the five durations of the most recent
 * call in milliseconds.
 * The events are created by taot_create and owned by the handle.
 * on = 1: the events only (the kernels are the ones an unprofiled call runs); on = 2: the matching + auction
 * kernel also counts cycles per part (taot_get_match_cycles), which slows it down; on = 3: taot_plan keeps its
 * layer groups (see taot_get_group_trace) and records the stage events per group instead.
 */
int taot_set_profiling(taot_handle_t h, int32_t on);
int taot_get_stage_ms(taot_handle_t h, float* h_ms /* [5] */);

/*
 * Timeline of the layer groups of the last taot_plan call made with profiling level 3 (a measurement aid; the
 * paper has no counterpart).  For a routing table large enough to be bandwidth-bound, taot_plan splits the L
 * problems into up to 6 groups of consecutive layers and plans each on a stream of its own, so that the
 * histogram and reassignment of one group run under the Sinkhorn and auction rounds of another; results are
 * those of an unsplit call.  *groups receives the number of groups (0: the handle does not split), h_ms
 * [groups][6] the time in ms, from the start of the call, at which each group reached: start, end of chunk
 * histogram, merge, Sinkhorn, matching + auction, reassignment.  Waits for the call to finish.
 * The environment variable TAOT_PLAN_GROUPS (read by taot_create) caps the number of groups; 1 disables the split.
 */
int taot_get_group_trace(taot_handle_t h, int32_t* groups, float* h_ms /* [6][6] */);


/*
 * Where the matching + auction kernel spends its time (a measurement aid; the paper has no counterpart).
 * With profiling level 2 (taot_set_profiling), taot_match / taot_plan make the kernel count SM clock cycles, as thread 0 of each layer's
 * CTA sees them, into `ws`; this call copies them to the host (it synchronises the device).
 *   h_cycles [L][16]: 0 set-up (loads, spill, round-invariant score terms), 1 Phase 2 (Algorithm 2),
 *   2 set-up of Phase 3, 3 Phase-3 bids (round start to the barrier after arbitration, summed over rounds),
 *   4 Phase-3 updates (to the barrier that ends the round), 5 the whole kernel, 6 / 7 the probe and the
 *   arbitration time of the thread that spent most on each (its own time, no waiting at barriers),
 *   8-11 Phase 2 split: rank scans + arbitration, winners, re-forming the served experts' keys, forming all keys
 *   once per slot index; 12 the Phase-3 loop as a whole (3 and 4 are what thread 0 sees between its own clock reads:
 *   loads of the next round that the compiler starts before the round's first clock read fall outside them, and the
 *   counting build itself is slower than the timed one, so 12 / rounds is an upper bound per round); 13-15 zero.
 * `ws` is the workspace of the profiled call.  Errors: TAOT_ERR_NULL, TAOT_ERR_UNSUPPORTED (R > 256).
 */
int taot_get_match_cycles(taot_handle_t h, const void* ws, int64_t* h_cycles /* [L][16] */);

/*
 * Arithmetic ceilings of the current device, measured: FP32 fused multiply-add throughput (TFLOP/s, 2 flops per
 * FMA) and ex2 special-function throughput (T op/s).  They are the denominators of the Sinkhorn stage's roofline
 * (its inner loop is FP32 multiply-adds; its log-domain steps are ex2/lg2).  (The paper has no counterpart: a
 * measurement aid, not a step of the method.)  Launches two register-only kernels five times each on `stream`,
 * WAITS for them, and returns the best rate.  d_sink: device memory of at least 4 * 2048 * (number of SMs) bytes
 * (practically never written).  h_*: host floats.  Errors: TAOT_ERR_NULL, TAOT_ERR_CUDA.
 */
int taot_measure_alu_peaks(float* h_fma_tflops, float* h_ex2_tops, void* d_sink, void* stream);

/*
 * Latencies of the current device, measured, in SM clock cycles per dependent operation: h_cycles[0] one level of
 * a warp shuffle reduction (shfl.xor + add), [1] one FP32 fused multiply-add, [2] one scaling update (rcp.approx +
 * multiply-add).  With few problems per call the Sinkhorn stage is one dependent chain per problem: the sum of
 * these latencies along one iteration is the floor its iteration time is compared with.  (The paper has no
 * counterpart: a measurement aid, not a step of the method.)  Launches one warp on `stream` and WAITS for it.
 * d_sink: device memory of at least 16 bytes (overwritten).  h_cycles: host floats [3].
 * Errors: TAOT_ERR_NULL, TAOT_ERR_CUDA.
 */
int taot_measure_latencies(float* h_cycles /* [3] */, void* d_sink, void* stream);

/*
 * Latencies of the operations a round of the Phase-3 auction (Algorithm 3) is a chain of, measured on the current
 * device in SM clock cycles, the way the matching kernel uses them (one CTA of eight warps): h_cycles[0] a dependent
 * shared-memory load, [1] a shared-memory atomicMax whose result is waited for, [2] a named barrier over the eight
 * warps, [3] the arbitration triple as a unit (atomicMax into a word, barrier, read-back of the word).  A round is
 * probe (load), arbitration (triple), update (atomic, load) and the closing barrier: their sum is the floor the
 * measured time per round is compared with.  (The paper has no counterpart: a measurement aid, not a step of the
 * method.)  Launches one CTA on `stream` and WAITS for it.  d_sink: device memory of at least 32 bytes (overwritten).
 * h_cycles: host floats [4].  Errors: TAOT_ERR_NULL, TAOT_ERR_CUDA.
 */
int taot_measure_round_latencies(float* h_cycles /* [4] */, void* d_sink, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TAOT_MEASURE_H */
