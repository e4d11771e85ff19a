/*
 * taot.h -- C ABI of the TAOT replica-placement planner for one NVIDIA B200 (sm_100a).
 *
 * The planner turns one micro-batch of MoE router decisions into an executable guest-replica
 * schedule.  Per problem (one MoE layer x one micro-batch; L problems per call, all
 * independent) it runs, on the GPU and without ever returning to the host:
 *
 *   taot_histogram      token loads n[r][e], per-expert and per-rank loads   (Appendix A.1)
 *   taot_excess_spare   overload / spare capacity against the integer mean   (Appendix A.1)
 *   taot_sinkhorn       Phase 1: entropic OT by Sinkhorn-Knopp over the rank-by-rank topology
 *                       cost, giving the flow hint T                         (Appendix A.2)
 *   taot_match          Phase 2: column-priority integer replica matching    (Appendix A.3, Alg. 2)
 *                       Phase 3: Lagrangian auction, rank -> slot counts X   (Appendix A.4, Alg. 3)
 *   taot_assign         deterministic token -> replica rewrite of the routing table
 *   taot_plan           all of the above chained on one stream
 *   taot_plan_host      taot_plan with host buffers (copies in and out on the same stream)
 *   taot_report         the per-layer dispatch diagnostics of a finished plan        (Appendix B.3)
 *   taot_dispatch       send counts and send-buffer positions for the token all-to-all that follows
 *
 * Conventions
 *   - Shapes: L problems, R ranks, E experts, K guest slots per rank, S = R*K slots
 *     (slot s = r*K + kappa lives on rank s / K), router top-k = k, T tokens per problem,
 *     T % R == 0; source rank of token t is t / (T/R).  All arrays are dense, row-major,
 *     in the index order written next to them.
 *   - Every pointer named d_* is DEVICE memory owned by the caller; h_* is HOST memory owned by
 *     the caller.  The library allocates device memory only inside taot_create (a few copies of
 *     the topology) and frees it in taot_destroy; scratch space is the caller's `ws`
 *     (taot_workspace_bytes bytes, 256-byte aligned).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     enqueue work and return; they never synchronise (except taot_create / taot_destroy).
 *   - Return value: TAOT_OK, or a negative taot_status found on the host before anything was
 *     launched.  Data-dependent conditions never fault or trap: they are OR-ed into d_info[l]
 *     (TAOT_INFO_* bits).  The caller zeroes d_info before the first stage it runs; taot_plan
 *     and taot_plan_host zero it themselves.
 *   - Same inputs give the same output bits on every call.
 */
#ifndef TAOT_H
#define TAOT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct taot_handle_s* taot_handle_t;

typedef enum {
    TAOT_OK = 0,
    TAOT_ERR_NULL = -1,         /* a required pointer is NULL */
    TAOT_ERR_PARAM = -2,        /* a parameter is out of its documented range */
    TAOT_ERR_UNSUPPORTED = -3,  /* a size is valid but beyond what this build supports */
    TAOT_ERR_CUDA = -4,         /* a CUDA runtime call failed (see cudaGetLastError) */
    TAOT_ERR_ALIGN = -5,        /* a device pointer is not aligned as required */
    TAOT_ERR_STATIC_CAPACITY = -6 /* the problem needs more than the built-in scratch of taot_histogram_static */
} taot_status;

/* bits of d_info[l] */
enum {
    TAOT_INFO_BAD_INDEX = 1,        /* topk_idx held a value outside [0, E): skipped / copied through */
    TAOT_INFO_SINKHORN_CAP = 2,     /* tolerance mode reached max_iters above tol */
    TAOT_INFO_NONFINITE = 4,        /* a non-finite value in the Sinkhorn solve, or in the s / d given to taot_sinkhorn */
    TAOT_INFO_AUCTION_RESIDUAL = 8, /* the auction stopped at auction_max_rounds with tokens unplaced */
    TAOT_INFO_SUPPLY_SCALED = 16,   /* sum(s) > sum(d): supply was scaled by gamma < 1 */
    TAOT_INFO_SINKHORN_SIZE = 32,   /* |hot| * |cold| exceeds the on-chip capacity: plan left at zero */
    TAOT_INFO_INTERNAL = 64         /* a bounded wait inside a kernel ran out (asynchronous copy never landed):
                                       the outputs of that call are incomplete */
};

/*
 * Problem description.  Set struct_size = sizeof(taot_params).
 * Supported ranges: 1 <= R <= 256 for the whole path (taot_excess_spare and taot_sinkhorn alone accept
 * R up to 1024; the other calls then return TAOT_ERR_UNSUPPORTED), 1 <= E <= 1024, 1 <= K <= 8,
 * 1 <= k <= 64, L >= 1, T >= R, T % R == 0, T*k < 2^31.
 */
typedef struct {
    int32_t struct_size;
    int32_t L;                  /* problems per call */
    int32_t R;                  /* expert-parallel ranks */
    int32_t E;                  /* experts */
    int32_t K;                  /* guest slots per rank */
    int32_t k;                  /* router top-k */
    int64_t T;                  /* tokens per problem */
    float   eps;                /* entropic regulariser (absolute, same unit as C), > 0 */
    int32_t max_iters;          /* Sinkhorn iterations if tol <= 0, iteration cap otherwise; >= 1 */
    float   tol;                /* stop once sum_i |rowsum_i - s~_i| <= tol * sum(s~); <= 0: fixed count */
    int32_t check_every;        /* test the tolerance every this many iterations (>= 1) */
    float   eps0;               /* the paper's epsilon_0 safeguard constant, e.g. 1e-8f */
    float   price_step;         /* Phase-3 price increment, e.g. 0.1f */
    int32_t auction_max_rounds; /* <= 0: run the auction to completion */
    int32_t ablation;           /* TAOT_ABLATE_* bits, 0 = the full method */
} taot_params;

/*
 * The two switches of the paper's algorithm-level ablation (Ablation Study, Table 2).  A term that is
 * switched off is left out of the Phase-2 score (which is the same as the term being exactly zero).
 * Phase 3 is never ablated: it only assigns tokens and always uses the real topology preference.
 */
enum {
    TAOT_ABLATE_HINT = 1,       /* no Phase-1 flow hint: taot_match ignores d_plan (it may be NULL); taot_plan does
                                   not run the Sinkhorn stage and returns a zero plan, zero iterations, zero row_err */
    TAOT_ABLATE_TOPOLOGY = 2    /* no topology-preference term alpha*B in the Phase-2 score */
};

/* Outputs of taot_plan / taot_plan_host: device pointers (host pointers for the _host call).
 * Optional members may be NULL and are then kept in workspace only. */
typedef struct {
    int32_t* n;             /* [L,R,E]   tokens rank r sends to expert e */
    int32_t* expert_load;   /* [L,E] */
    int32_t* rank_load;     /* [L,R] */
    int32_t* excess;        /* [L,R]     optional */
    int32_t* spare;         /* [L,R]     optional */
    float*   plan;          /* [L,R,R]   Phase-1 flow hint T, in tokens */
    int32_t* sinkhorn_iters;/* [L] */
    float*   row_err;       /* [L]       relative row-marginal violation at the returned iterate */
    int32_t* slot_expert;   /* [L,R,K]   expert placed in slot (r, kappa), -1 = empty */
    int32_t* slot_tokens;   /* [L,R,K]   tokens planned for that slot (the paper's A_es) */
    int32_t* X;             /* [L,R,S]   tokens source rank r sends to slot s */
    int32_t* rounds;        /* [L,2]     optional: Phase-2 inner rounds, Phase-3 rounds */
    int32_t* new_idx;       /* [L,T,k]   rewritten routing table: e, or E + s for a guest slot */
    int32_t* info;          /* [L]       TAOT_INFO_* bits */
} taot_outputs;

/*
 * Create a planner for a fixed topology.  (Problem Formulation: R, E, home ranks r_e, cost W.)
 *   h_e2r [E]   home rank of each expert, each in [0, R)
 *   h_C  [R,R]  communication cost from row rank to column rank, finite, >= 0
 *   h_B  [R,R]  topology preference (Appendix A.3: 1 intra-node, w_inter < 1 inter-node, 0 home),
 *               or NULL to derive it from C: B_ii = 0, B_ij = min(1, c_min / C_ij) with c_min the
 *               smallest positive off-diagonal cost (1 where C_ij <= 0).
 * All three are HOST arrays, copied during the call (which synchronises the device).
 * Errors: TAOT_ERR_NULL, TAOT_ERR_PARAM (ranges above, bad e2r entry, non-finite cost, eps <= 0),
 * TAOT_ERR_UNSUPPORTED, TAOT_ERR_CUDA.  On error *out is NULL.
 */
int taot_create(taot_handle_t* out, const taot_params* params, const int32_t* h_e2r,
                const float* h_C, const float* h_B);

/* Frees the handle's device copies.  Synchronises the device.  NULL is accepted. */
int taot_destroy(taot_handle_t h);

/* Scratch bytes taot_* calls need in `ws` for this handle (device memory, 256-byte aligned).  With at most 256
 * experts this includes L*T*k bytes for a one-byte copy of the routing table (see taot_assign). */
int taot_workspace_bytes(taot_handle_t h, size_t* bytes);

/* Device scratch bytes taot_plan_host needs (staging of inputs/outputs plus the workspace). */
int taot_host_workspace_bytes(taot_handle_t h, size_t* bytes);

/*
 * Load collection (Appendix A.1: n_re, and l_r = sum over r's experts of sum_r' n_r'e).
 *   d_topk [L,T,k] int32, 4-byte aligned (16-byte alignment enables the vector path).
 *   d_n [L,R,E], d_expert_load [L,E], d_rank_load [L,R]: fully overwritten.
 * Side effect: per-chunk counts stay in `ws` for a later taot_assign(..., reuse_counts = 1).
 * An index outside [0, E) is skipped and sets TAOT_INFO_BAD_INDEX.
 */
int taot_histogram(taot_handle_t h, const int32_t* d_topk, int32_t* d_n, int32_t* d_expert_load,
                   int32_t* d_rank_load, int32_t* d_info, void* ws, void* stream);

/*
 * taot_histogram for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a packaging variant of the load collection above, not a step of the method.)
 *
 * Who needs it: code that runs inside a memory plan it does not own -- a plug-in of a serving or
 * training runtime that has pre-carved all device memory, a stage called while its stream is being
 * captured, a process whose pool is exhausted.  Such a caller cannot cudaMalloc a workspace (the
 * call may fail, it synchronises the device, and it is not allowed during capture) and may not
 * have one to spare.  This entry point needs no handle and no workspace and calls no allocating
 * routine: the per-chunk counts it needs live in a fixed 256-byte-aligned device array of
 * TAOT_STATIC_SCRATCH_BYTES that is part of the library image.  Every GPU on which the library is
 * loaded holds that array until the process exits.
 *
 *   d_topk [L,T,k], d_e2r [E] (home rank of each expert, values in [0,R); an entry outside that range is
 *   caught on the device: the expert is left out of d_rank_load and TAOT_INFO_BAD_INDEX is set),
 *   d_n [L,R,E], d_expert_load [L,E], d_rank_load [L,R], d_info [L]: device memory of the caller,
 *   same meaning, layout and overwrite rules as taot_histogram; d_info is OR-ed into.
 *
 * Limits and rules:
 *   - L * R * ceil((T/R)*k / 16384) * E * 4 bytes must fit in TAOT_STATIC_SCRATCH_BYTES, otherwise
 *     nothing is launched and TAOT_ERR_STATIC_CAPACITY is returned.  Other errors as taot_histogram.
 *   - The first call on each device looks up the array's device address (with that device current).
 *     Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.  Each
 *     call overwrites every count it later reads, so nothing needs clearing; but two calls whose
 *     kernels overlap on the GPU (different streams, no dependency between them) race on it and
 *     give wrong loads.  Serialise them.
 *   - The per-chunk counts are not available to taot_assign afterwards (use reuse_counts = 0).
 */
#define TAOT_STATIC_SCRATCH_BYTES (4u << 20)
int taot_histogram_static(const int32_t* d_topk, int32_t L, int64_t T, int32_t k, int32_t R, int32_t E,
                          const int32_t* d_e2r, int32_t* d_n, int32_t* d_expert_load,
                          int32_t* d_rank_load, int32_t* d_info, void* stream);

/*
 * Excess / spare (Appendix A.1) against the integer mean m = floor(sum_r l_r / R), for B rows:
 *   excess = max(l - m, 0), spare = max(m - l, 0); d_s / d_d receive the same as fp32
 *   (the supply and demand vectors of Phase 1).  Any output pointer may be NULL.
 */
int taot_excess_spare(taot_handle_t h, const int32_t* d_rank_load, int32_t B, int32_t* d_excess,
                      int32_t* d_spare, float* d_s, float* d_d, void* stream);

/*
 * Phase 1 (Appendix A.2).  For each of B problems: supply d_s[b,:], demand d_d[b,:] (fp32, >= 0),
 * cost C and eps from the handle.  gamma = min(1, sum d / max(sum s, eps0)), s~ = gamma s;
 * iterate u = s~/(M v), v = d/(M^T u) from v = 1, M = exp(-C/eps), for max_iters iterations or
 * until the row-marginal test passes; T = diag(u) M diag(v) followed by the column cap
 * T_ij *= min(1, d_j / (sum_i T_ij + eps0)).
 *   d_plan [B,R,R] fp32 (fully overwritten), d_iters [B], d_row_err [B], d_info [B].
 * The iterates are carried so that neither M nor u, v can under- or overflow for any C/eps.
 * `ws` is needed only for R > 256 (the kernel matrix then lives in workspace; batches larger than
 * the handle's L are solved in slices of L).  Problems with |{s>0}| * |{d>0}| beyond the capacity
 * (R*R/4 for R > 128, which disjoint supply/demand ranks never exceed) get TAOT_INFO_SINKHORN_SIZE
 * and a zero plan.
 * Kernel choice (all give the same iterates up to fp32 rounding): a cost that depends only on the tier of a rank
 * pair (same node / same rail group / neither; see taot_tier_structure) at 256, 512 or 1024 ranks is summed tier by tier; up to
 * 256 ranks the kernel matrix of a problem lives in registers or shared memory; beyond 256 ranks a batch of at least
 * 256 problems with a fixed iteration count (tol <= 0) and max(C)/eps <= 20 is solved as dense products
 * [R,R] x [R,B] on the tensor cores (tcgen05, three TF32 products per term; the row error it reports is the true row
 * violation of the returned plan, a few 1e-6 of the total mass from accumulator truncation), anything else beyond
 * 256 ranks by four-CTA clusters.  Environment, read at taot_create / at the call: TAOT_NO_TENSOR_CORES (any value)
 * keeps the dense path off, TAOT_TC_TILE_N = 64 | 128 | 256 forces its tile width.
 * A problem whose s or d holds a NaN or an infinity gets TAOT_INFO_NONFINITE, a zero
 * plan and 0 iterations; the other problems of the batch are not affected.
 */
int taot_sinkhorn(taot_handle_t h, const float* d_s, const float* d_d, int32_t B, float* d_plan,
                  int32_t* d_iters, float* d_row_err, int32_t* d_info, void* ws, void* stream);

/*
 * Phases 2 and 3 (Appendix A.3 / Algorithm 2, Appendix A.4 / Algorithm 3) for L problems.
 * Spill comes from d_expert_load by cumulative-excess differencing within each rank; the score
 * min(spill, spare) + alpha B + 0.1 alpha T_norm (alpha = m R / E) is evaluated in fp32 with one
 * rounding per operation; both argmax ties go to the lowest index.
 *   in : d_n [L,R,E], d_expert_load [L,E], d_rank_load [L,R], d_plan [L,R,R]
 *   out: d_slot_expert [L,R,K], d_slot_tokens [L,R,K], d_X [L,R,S], d_rounds [L,2] (or NULL)
 */
int taot_match(taot_handle_t h, const int32_t* d_n, const int32_t* d_expert_load,
               const int32_t* d_rank_load, const float* d_plan, int32_t* d_slot_expert,
               int32_t* d_slot_tokens, int32_t* d_X, int32_t* d_rounds, int32_t* d_info, void* ws,
               void* stream);

/*
 * Token reassignment (Problem Formulation: the paper leaves the per-token rule open and fixes only
 * the counts X; the rule here is earliest entries first, lowest slot first).  Within each
 * (source rank, expert) group, in flat order t*k + j, the slots holding that expert take, lowest
 * slot first, the first X[r][s] entries; an entry so taken is rewritten to E + s, the rest keep e.
 *   d_new_idx [L,T,k] must not alias d_topk.
 *   reuse_counts != 0: trust what taot_histogram left in `ws` for the same d_topk -- the per-chunk counts and, with at
 *   most 256 experts, 16-byte aligned tables and rank segments of a multiple of 16 entries, a copy of the table as one
 *   byte per entry with one flag per chunk, which the rewrite then reads instead of d_topk (chunks holding a value that
 *   is no expert are read from d_topk itself); 0: recount (one more read of d_topk).
 */
int taot_assign(taot_handle_t h, const int32_t* d_topk, const int32_t* d_slot_expert,
                const int32_t* d_X, int32_t* d_new_idx, int32_t* d_info, void* ws,
                int32_t reuse_counts, void* stream);

/*
 * The whole path (Algorithm 1: Phase 1, Phase 2, Phase 3, then the rewrite), asynchronous on `stream`; `out` holds
 * DEVICE pointers.  No allocation, no synchronisation: the call can be captured in a CUDA graph.
 * A routing table large enough to be bandwidth-bound (more than three waves of chunks per part) is planned in up to
 * six groups of consecutive layers: group 0 on `stream`, the others on streams the handle created, forked from
 * `stream` by an event and joined back into it by events before the call returns control to `stream`'s order; the
 * results are those of an unsplit call, bit for bit.  (The histogram and reassignment of one group then run under
 * the Sinkhorn and auction rounds of another.)  TAOT_PLAN_GROUPS (environment, read by taot_create) caps the number
 * of groups; 1 keeps everything on `stream`.
 */
int taot_plan(taot_handle_t h, const int32_t* d_topk, const taot_outputs* out, void* ws, void* stream);

/*
 * The whole path with HOST buffers: h_topk [L,T,k] is copied to the device, the path runs, and
 * every non-NULL member of `out` (HOST pointers) is copied back, all enqueued on `stream`.
 * Pinned host memory makes the copies asynchronous.  d_ws: taot_host_workspace_bytes bytes.
 */
int taot_plan_host(taot_handle_t h, const int32_t* h_topk, const taot_outputs* out, void* d_ws,
                   void* stream);

/*
 * taot_plan_host with the results packed: the rewritten routing table goes to h_new_idx [L,T,k] and EVERY other
 * member of taot_outputs to one host block, in two device-to-host copies instead of one per output (a small copy
 * costs the copy engine about as much as 0.5 MB does, which bounds throughput when several calls are in flight).
 * taot_host_block_layout gives the block's size and, in the order of taot_outputs' members, the byte offset of every
 * output inside it (multiples of 256; the entry of new_idx, member 12, is SIZE_MAX).  Bytes between outputs are
 * overwritten.  Pinned host memory makes the copies asynchronous.  d_ws: taot_host_workspace_bytes bytes.
 * Errors: TAOT_ERR_NULL, TAOT_ERR_ALIGN, and those of taot_plan.
 */
int taot_host_block_layout(taot_handle_t h, size_t* offsets /* [14] */, size_t* bytes);
int taot_plan_host_block(taot_handle_t h, const int32_t* h_topk, int32_t* h_new_idx, void* h_block, void* d_ws,
                         void* stream);

/*
 * Dispatch metadata for the token all-to-all that follows the planner (Method: the rewritten routing is what the
 * dispatcher executes; the paper does not spell the bookkeeping out, so the layout below is this library's).
 * For each problem l and source rank r (the R contiguous segments of (T/R)*k entries of d_new_idx[l]):
 *   d_send_counts [L,R,R]      [l][r][q] = entries of source rank r that execute on rank q
 *                              (target e < E executes on its home rank, target E + s on rank s / K)
 *   d_target_counts [L,R,E+S]  [l][r][t] = entries of source rank r with target t; optional (NULL to skip)
 *   d_perm [L,T,k]             position of every entry in its source rank's send buffer when that buffer is ordered
 *                              by (destination rank, target index, original flat order): a stable sort, so
 *                              send_buffer[perm[i]] = entry i; positions run over [0, (T/R)*k) per source rank
 * An index outside [0, E+S) cannot be delivered: it is counted nowhere, its positions follow all valid entries in
 * original order, and TAOT_INFO_BAD_INDEX is set.  d_perm must not alias d_new_idx.  Uses `ws`.
 * Errors: TAOT_ERR_NULL, TAOT_ERR_ALIGN (4-byte tables, 256-byte ws), TAOT_ERR_PARAM (aliasing),
 * TAOT_ERR_UNSUPPORTED (R > 256).
 */
int taot_dispatch(taot_handle_t h, const int32_t* d_new_idx, int32_t* d_send_counts, int32_t* d_target_counts,
                  int32_t* d_perm, int32_t* d_info, void* ws, void* stream);

/*
 * One layer's dispatch diagnostics (Appendix B.3; metric definitions of the Evaluation section).  128 bytes.
 */
typedef struct {
    int64_t total_load;      /* sum_r l_r */
    int64_t rerouted;        /* sum_{r,s} X[r][s]: tokens sent to guest replicas */
    int32_t mean_load;       /* floor(total_load / R), the mean the planner balances against */
    int32_t max_before, min_before;   /* extreme rank loads before rerouting */
    int32_t max_after, min_after;     /* extreme projected rank loads after rerouting */
    int32_t hot_ranks;       /* ranks with l_r above the mean */
    int32_t cold_ranks;      /* ranks with l_r below the mean */
    int32_t hot_experts;     /* experts with positive spill (the candidates of Phase 2) */
    int32_t clones;          /* occupied guest slots = expert-weight transfers */
    int32_t intra, inter;    /* of those: inside the home node (B[home][host] >= 1) / across nodes */
    int32_t same_rank;       /* of those: hosted by the home rank itself (neither intra nor inter) */
    double rho_before, rho_after;     /* (max_r l_r - mean) / mean with mean = total_load / R */
    double dev_before, dev_after;     /* max_r |l_r - mean| / mean */
    double peak_reduction;   /* (max_before - max_after) / max_before */
    double frac_rerouted;    /* rerouted / total_load */
    double cost_ratio;       /* intra + lambda * inter: the weighted cost at 1 : lambda */
    double cost_C;           /* sum over occupied slots of C[home rank][host rank] */
} taot_report_row;

/*
 * Dispatch report of L finished plans (Appendix B.3, parts 1-4), computed on the GPU.
 *   in : d_expert_load [L,E], d_rank_load [L,R], d_slot_expert [L,R,K], d_X [L,R,S] as taot_plan wrote them;
 *        lambda: the inter-node weight of cost_ratio (the paper uses 3).
 *   out: d_rows [L] (device memory, 8-byte aligned); optional (NULL to skip) per-element arrays
 *        d_spill [L,E]        spill of each expert before matching (part 1: the hot experts are spill > 0)
 *        d_load_after [L,R]   projected rank loads (part 3)
 *        d_slot_moved [L,S]   tokens rerouted to each slot (part 2)
 *        d_slot_kind [L,S]    0 empty, 1 intra-node copy, 2 inter-node copy, 3 hosted by the home rank
 * Integer fields are exact; each ratio is a single IEEE fp64 operation; a zero denominator gives 0.
 * A zero ratio or an empty plan is not an error.  Errors: TAOT_ERR_NULL, TAOT_ERR_ALIGN,
 * TAOT_ERR_UNSUPPORTED (R > 256), TAOT_ERR_PARAM (lambda not finite).
 */
int taot_report(taot_handle_t h, const int32_t* d_expert_load, const int32_t* d_rank_load,
                const int32_t* d_slot_expert, const int32_t* d_X, double lambda, taot_report_row* d_rows,
                int32_t* d_spill, int32_t* d_load_after, int32_t* d_slot_moved, int32_t* d_slot_kind,
                void* stream);

/*
 * The hierarchy taot_create found in the cost matrix (Appendix A.1 builds W from node membership): if C depends
 * only on whether two ranks share a node, share a rail group of nodes, or neither, with block sizes the tier-by-tier
 * Sinkhorn kernels are built for (ranks per node / per group: 8 / 32, 4 / 16, 4 / 32, 16 / 32; 256, 512 or 1024
 * ranks), *node and *group receive those sizes; otherwise both are 0 and the kernels that hold the kernel matrix run.
 */
int taot_tier_structure(taot_handle_t h, int32_t* node, int32_t* group);

/* Kernels launched by the last call on this handle (for launch accounting). */
int taot_last_launch_count(taot_handle_t h, int32_t* count);

const char* taot_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* TAOT_H */
