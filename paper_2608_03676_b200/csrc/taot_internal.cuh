// Internal definitions shared by the translation units of libtaot (never installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "taot.h"
#include "taot_measure.h"

// Elements of topk_idx one CTA of the histogram / reassignment kernels owns.  A chunk never
// crosses a (layer, source rank) segment, so a segment of SEG = (T/R)*k elements has
// NC = ceil(SEG / TAOT_CHUNK) chunks, the last one possibly short.
#define TAOT_CHUNK 16384
#define TAOT_STREAM_THREADS 256            // threads of the streaming kernels: 64 elements each
#define TAOT_MAX_TIERS 8                   // distinct bonus values the bit-set auction handles
#define TAOT_MERGE_PARTS 8                 // CTAs that share the merge of one layer's chunk counts (256-rank tables)
#define TAOT_MAX_GROUPS 6                  // layer groups taot_plan overlaps on internal streams

struct taot_handle_s {
    taot_params p;
    int device;
    int sm_count;
    // topology, device copies
    int32_t* d_e2r;          // [E]
    float* d_C;              // [R,R]
    float* d_B;              // [R,R] topology preference (given or derived)
    double* d_rowlse0;       // [R]  LSE_j(-C_ij/eps) over all ranks j: the first u-update with v = 1
    float* d_gibbs;          // [4][R,R] exp(-C/eps) and its transpose, each as TF32-exact high and low parts (tensor-core
                             // solve: more than 256 ranks, no tier structure, max C/eps <= 20), else null
    int32_t* d_rank_off;     // [R+1] CSR of experts by home rank
    int32_t* d_rank_list;    // [E]
    uint32_t* d_tiermask;    // [ntiers][W][R hosts] bit r of word w set iff bonus(32w + r -> host) == tierval[t]; null if ntiers == 0
    int32_t* d_tpos;         // [E+S+1] position of each target in (destination rank, target) order; last = undeliverable
    int32_t* d_torder;       // [E+S+1] target at each position
    int32_t* d_tdest;        // [E+S+1] destination rank of each target (R for the undeliverable bin)
    float* d_tierval;        // [ntiers] distinct values of the auction bonus matrix, descending
    int32_t ntiers;          // 0: too many distinct values, the auction scans densely
    uint32_t* d_bidlist;     // [nbid] every (tier, win count) pair, best score first: w << 8 | t, bit 31 = next has the same score
    int32_t nbid;            // 0: no list (no tiers, or price step <= 0): the auction scans densely
    int32_t* d_merge_part;   // [L][TAOT_MERGE_PARTS][E] expert loads of the parts of a layer's merge, or null (one CTA per layer)
    int32_t* d_merge_cnt;    // [L] parts of a layer's merge that are done; zero between calls
    int32_t tier_ok;         // 1: C has a node / rail-group structure one of the tier-by-tier kernels is built for and R is 256, 512 or 1024
    int32_t tier_node, tier_group;   // ranks per node and per rail group of that structure (8 / 32, 4 / 16, 4 / 32 or 16 / 32)
    float tier_cost[3];      // its three costs off the diagonal: same node, same rail group, otherwise
    // derived sizes
    int64_t seg;             // elements per (layer, rank) segment
    int32_t nc;              // chunks per segment
    int32_t kcap;            // Sinkhorn kernel-matrix capacity in floats per problem (shared memory)
    int64_t kcap_global;     // same, global-memory scratch per problem (R > 256 only), else 0
    // workspace layout (byte offsets)
    size_t off_cc, off_excess, off_spare, off_s, off_d, off_nrem, off_t12, off_kt, off_dc, off_cyc, off_tc;
    size_t off_tb, off_tbflag;   // one-byte copy of the routing table and one flag per chunk (see tb_ok)
    int32_t tb_ok;               // 1: the histogram pass also leaves the table as one byte per entry (E <= 256 experts,
                                 // segments of a multiple of 16 entries) for the reassignment to read instead of the table
    size_t ws_bytes;
    // host-call staging layout (byte offsets into d_ws of taot_plan_host)
    size_t hoff_topk, hoff_new, hoff_n, hoff_el, hoff_rl, hoff_ex, hoff_sp, hoff_plan, hoff_it, hoff_err,
           hoff_se, hoff_st, hoff_X, hoff_rounds, hoff_info, hoff_ws;
    size_t host_ws_bytes;
    int32_t last_launches;
    int32_t profiling;
    cudaEvent_t ev[6];
    // Layer groups of taot_plan (large routing tables only): group g is a view of this handle on layers
    // [group_l0[g], group_l0[g] + group[g]->p.L) -- same topology pointers, workspace offsets moved to the group's
    // first layer -- planned on a stream of its own so that the bandwidth-bound stages of one group run under the
    // latency-bound stages of another.  ngroups <= 1: one group on the caller's stream.
    int32_t is_view;                           // a view owns nothing
    int32_t ngroups;
    taot_handle_s* group[TAOT_MAX_GROUPS];
    int32_t group_l0[TAOT_MAX_GROUPS];
    int32_t group_len[TAOT_MAX_GROUPS];
    cudaStream_t gstream[TAOT_MAX_GROUPS];     // [0] unused: group 0 runs on the caller's stream
    cudaEvent_t ev_fork, ev_hist[TAOT_MAX_GROUPS], ev_join[TAOT_MAX_GROUPS];
    cudaStream_t bstream;                      // the one-byte copies of the groups' tables are made here, after all histograms
    cudaEvent_t ev_bytes[TAOT_MAX_GROUPS];     // group g's copy is there
};

static inline size_t taot_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// kernel launchers (each returns the number of kernels it enqueued, or a negative taot_status)
int taot_launch_histogram(taot_handle_t h, const int32_t* d_topk, int32_t* d_cc, int32_t* d_info, cudaStream_t st,
                          void* ws = nullptr, bool write_bytes = true);
// the table as one byte per entry, by a few CTAs that leave the other SMs alone (returns 0 if this handle keeps no such copy)
int taot_launch_table_bytes(taot_handle_t h, const int32_t* d_topk, void* ws, cudaStream_t st);
int taot_launch_merge(taot_handle_t h, const int32_t* d_cc, int32_t* d_n, int32_t* d_expert_load,
                      int32_t* d_rank_load, int32_t* d_excess, int32_t* d_spare, float* d_s, float* d_d,
                      cudaStream_t st, int32_t* d_info = nullptr);
int taot_launch_excess_spare(taot_handle_t h, const int32_t* d_rank_load, int32_t B, int32_t* d_excess,
                             int32_t* d_spare, float* d_s, float* d_d, cudaStream_t st);
int taot_launch_sinkhorn(taot_handle_t h, const float* d_s, const float* d_d, int32_t B, float* d_plan,
                         int32_t* d_iters, float* d_row_err, int32_t* d_info, float* d_kt, cudaStream_t st,
                         float* d_tc = nullptr);
size_t taot_sinkhorn_tc_ws_floats(int32_t R, int32_t B);
int taot_launch_sinkhorn_guard(taot_handle_t h, const float* d_s, const float* d_d, int32_t B, float* d_plan,
                               int32_t* d_iters, float* d_row_err, int32_t* d_info, cudaStream_t st);
int taot_launch_match(taot_handle_t h, const int32_t* d_n, const int32_t* d_expert_load,
                      const int32_t* d_rank_load, const float* d_plan, int32_t* d_slot_expert,
                      int32_t* d_slot_tokens, int32_t* d_X, int32_t* d_rounds, int32_t* d_info,
                      int32_t* d_nrem, float* d_t12, cudaStream_t st, long long* d_cyc = nullptr);
int taot_launch_assign(taot_handle_t h, const int32_t* d_topk, void* ws, const int32_t* d_slot_expert,
                       const int32_t* d_X, int32_t* d_new_idx, int32_t* d_info, cudaStream_t st);

int taot_launch_report(taot_handle_t h, const int32_t* d_expert_load, const int32_t* d_rank_load,
                       const int32_t* d_slot_expert, const int32_t* d_X, double lambda, taot_report_row* d_rows,
                       int32_t* d_spill, int32_t* d_load_after, int32_t* d_slot_moved, int32_t* d_slot_kind,
                       cudaStream_t st);

int taot_launch_chunk_counts(taot_handle_t h, const int32_t* d_idx, int32_t* d_counts, int32_t* d_info, int32_t bins,
                             cudaStream_t st);
int taot_launch_dispatch(taot_handle_t h, const int32_t* d_new_idx, int32_t* d_send_counts, int32_t* d_target_counts,
                         int32_t* d_perm, int32_t* d_info, void* ws, cudaStream_t st);

#define TAOT_CUDA_OK(expr)                              \
    do {                                                \
        cudaError_t _e = (expr);                        \
        if (_e != cudaSuccess) return TAOT_ERR_CUDA;    \
    } while (0)
