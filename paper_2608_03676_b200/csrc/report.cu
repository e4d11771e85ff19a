// Dispatch report (Appendix B.3: the per-layer diagnostics in four parts; Evaluation: imbalance,
// intra-/inter-node transfers and the weighted cost at 1 : lambda).  One CTA per layer; everything is
// small (R ranks, E experts, S slots), so the kernel is a handful of block-wide passes:
//   part 1  spill per expert (cumulative-excess differencing inside the home rank, by ranking each expert
//           among the experts of its rank), hot / cold rank and hot expert counts, max / min load
//   part 2  tokens rerouted to each slot (column sums of X), kind of each copy, counts, weighted costs
//   part 3  projected load per rank
//   part 4  imbalance before / after, largest deviation, peak reduction, fraction rerouted
// Integer results are exact; every ratio is one fp64 IEEE operation (explicit *_rn intrinsics, so nothing is
// contracted), and the fp64 cost sum runs over the slots in ascending order in one thread.
#include "taot_internal.cuh"

namespace {

constexpr int kThreads = 256;

struct ReportArgs {
    const int32_t* e2r;
    const int32_t* rank_off;
    const int32_t* rank_list;
    const float* C;
    const float* B;
    const int32_t* expert_load;   // [L,E]
    const int32_t* rank_load;     // [L,R]
    const int32_t* slot_expert;   // [L,S]
    const int32_t* X;             // [L,R,S]
    taot_report_row* rows;        // [L]
    int32_t* spill;               // [L,E] or null
    int32_t* load_after;          // [L,R] or null
    int32_t* slot_moved;          // [L,S] or null
    int32_t* slot_kind;           // [L,S] or null
    double lambda;
    int32_t R, E, K;
};

__device__ __forceinline__ long long block_sum(long long v, long long* red)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    long long t = 0;
    for (int w = 0; w < kThreads / 32; ++w) t += red[w];
    return t;
}

__device__ __forceinline__ int block_max(int v, long long* red)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    int t = (int)red[0];
    for (int w = 1; w < kThreads / 32; ++w) t = max(t, (int)red[w]);
    return t;
}

__global__ void __launch_bounds__(kThreads)
report_kernel(ReportArgs a)
{
    extern __shared__ int32_t sh[];
    const int R = a.R, E = a.E, K = a.K, S = R * K;
    int32_t* after = sh;            // [R]
    int32_t* moved = after + R;     // [S]
    int32_t* kind = moved + S;      // [S]
    __shared__ long long red[kThreads / 32];
    const int tid = threadIdx.x;
    const int64_t l = blockIdx.x;
    const int32_t* el = a.expert_load + l * E;
    const int32_t* rl = a.rank_load + l * R;
    const int32_t* se = a.slot_expert + l * S;
    const int32_t* X = a.X + l * (int64_t)R * S;

    // ---- part 1
    long long part = 0;
    int mx = INT32_MIN, mn_neg = INT32_MIN;
    for (int r = tid; r < R; r += kThreads) {
        const int v = rl[r];
        part += v; mx = max(mx, v); mn_neg = max(mn_neg, -v);
        after[r] = v;
    }
    const long long total = block_sum(part, red);
    const int max_b = block_max(mx, red);
    const int min_b = -block_max(mn_neg, red);
    const long long mfloor = total / R;
    long long hot_r = 0, cold_r = 0;
    for (int r = tid; r < R; r += kThreads) { hot_r += rl[r] > mfloor; cold_r += rl[r] < mfloor; }
    hot_r = block_sum(hot_r, red);
    cold_r = block_sum(cold_r, red);

    long long hot_e = 0;
    for (int e = tid; e < E; e += kThreads) {
        // cumulative load of the experts of e's rank that sort at or before e by (load, index)
        const int h = a.e2r[e];
        const int le = el[e];
        long long cum = 0;
        for (int q = a.rank_off[h]; q < a.rank_off[h + 1]; ++q) {
            const int o = a.rank_list[q];
            const int lo = el[o];
            if (lo < le || (lo == le && o <= e)) cum += lo;
        }
        const long long sig = cum > mfloor ? cum - mfloor : 0;
        const long long before = cum - le;
        const long long sig_prev = before > mfloor ? before - mfloor : 0;
        const int sp = (int)(sig - sig_prev);
        if (a.spill) a.spill[l * E + e] = sp;
        hot_e += sp > 0;
    }
    hot_e = block_sum(hot_e, red);

    // ---- part 2
    long long rer = 0, clones = 0, intra = 0, inter = 0, same = 0;
    for (int s = tid; s < S; s += kThreads) {
        long long m = 0;
        for (int r = 0; r < R; ++r) m += X[(int64_t)r * S + s];
        moved[s] = (int32_t)m;
        rer += m;
        const int e = se[s];
        int kd = 0;
        if (e >= 0 && e < E) {
            const int home = a.e2r[e], host = s / K;
            ++clones;
            if (home == host) { kd = 3; ++same; }
            else if (a.B[(int64_t)home * R + host] >= 1.0f) { kd = 1; ++intra; }
            else { kd = 2; ++inter; }
        }
        kind[s] = kd;
        if (a.slot_moved) a.slot_moved[l * S + s] = (int32_t)m;
        if (a.slot_kind) a.slot_kind[l * S + s] = kd;
    }
    rer = block_sum(rer, red);
    clones = block_sum(clones, red);
    intra = block_sum(intra, red);
    inter = block_sum(inter, red);
    same = block_sum(same, red);

    // ---- part 3 (integer adds: any order gives the same result)
    for (int s = tid; s < S; s += kThreads) {
        if (kind[s] == 0 || moved[s] == 0) continue;
        atomicSub(&after[a.e2r[se[s]]], moved[s]);
        atomicAdd(&after[s / K], moved[s]);
    }
    __syncthreads();
    mx = INT32_MIN; mn_neg = INT32_MIN;
    for (int r = tid; r < R; r += kThreads) {
        const int v = after[r];
        mx = max(mx, v); mn_neg = max(mn_neg, -v);
        if (a.load_after) a.load_after[l * R + r] = v;
    }
    const int max_a = block_max(mx, red);
    const int min_a = -block_max(mn_neg, red);

    // ---- part 4
    if (tid == 0) {
        double cost_C = 0.0;
        for (int s = 0; s < S; ++s)
            if (kind[s] != 0) cost_C = __dadd_rn(cost_C, (double)a.C[(int64_t)a.e2r[se[s]] * R + s / K]);
        taot_report_row o;
        o.total_load = total; o.rerouted = rer; o.mean_load = (int32_t)mfloor;
        o.max_before = max_b; o.min_before = min_b; o.max_after = max_a; o.min_after = min_a;
        o.hot_ranks = (int32_t)hot_r; o.cold_ranks = (int32_t)cold_r; o.hot_experts = (int32_t)hot_e;
        o.clones = (int32_t)clones; o.intra = (int32_t)intra; o.inter = (int32_t)inter; o.same_rank = (int32_t)same;
        const double mean = __ddiv_rn((double)total, (double)R);
        o.rho_before = o.rho_after = o.dev_before = o.dev_after = 0.0;
        if (mean > 0.0) {
            const double up_b = __dsub_rn((double)max_b, mean), dn_b = __dsub_rn(mean, (double)min_b);
            const double up_a = __dsub_rn((double)max_a, mean), dn_a = __dsub_rn(mean, (double)min_a);
            o.rho_before = __ddiv_rn(up_b, mean);
            o.rho_after = __ddiv_rn(up_a, mean);
            o.dev_before = __ddiv_rn(up_b > dn_b ? up_b : dn_b, mean);
            o.dev_after = __ddiv_rn(up_a > dn_a ? up_a : dn_a, mean);
        }
        o.peak_reduction = max_b > 0 ? __ddiv_rn((double)(max_b - max_a), (double)max_b) : 0.0;
        o.frac_rerouted = total > 0 ? __ddiv_rn((double)rer, (double)total) : 0.0;
        o.cost_ratio = __dadd_rn((double)intra, __dmul_rn(a.lambda, (double)inter));
        o.cost_C = cost_C;
        a.rows[l] = o;
    }
}

}  // namespace

int taot_launch_report(taot_handle_t h, const int32_t* d_expert_load, const int32_t* d_rank_load,
                       const int32_t* d_slot_expert, const int32_t* d_X, double lambda, taot_report_row* d_rows,
                       int32_t* d_spill, int32_t* d_load_after, int32_t* d_slot_moved, int32_t* d_slot_kind,
                       cudaStream_t st)
{
    const taot_params& p = h->p;
    ReportArgs a;
    a.e2r = h->d_e2r; a.rank_off = h->d_rank_off; a.rank_list = h->d_rank_list; a.C = h->d_C; a.B = h->d_B;
    a.expert_load = d_expert_load; a.rank_load = d_rank_load; a.slot_expert = d_slot_expert; a.X = d_X;
    a.rows = d_rows; a.spill = d_spill; a.load_after = d_load_after; a.slot_moved = d_slot_moved;
    a.slot_kind = d_slot_kind; a.lambda = lambda; a.R = p.R; a.E = p.E; a.K = p.K;
    const size_t smem = sizeof(int32_t) * ((size_t)p.R + 2 * (size_t)p.R * p.K);
    report_kernel<<<(unsigned)p.L, kThreads, smem, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
