// Dispatch metadata after the planner (what the token all-to-all that follows needs; the paper's system passes
// the rewritten routing to its dispatcher, Method / System Design).  For every source rank: how many of its
// entries execute on each rank, how many go to each target (expert or guest slot), and the position of every
// entry in the rank's send buffer ordered by (destination rank, target, original order) -- a stable counting
// sort with E + S keys, done as three passes over chunks of <= 16384 entries:
//   hist_chunk_kernel        (histogram.cu) one CTA per chunk: histogram of the chunk over the E + S targets,
//                            with one more bin for values that are no target
//   dispatch_offsets_kernel  one CTA per (layer, source rank): totals, exclusive scan in destination order,
//                            per-chunk bases (in place), send counts per destination rank
//   dispatch_scatter_kernel  one CTA per chunk: per-warp histograms of the warp's contiguous span, bases per
//                            warp, then each warp walks its span in order, 32 entries at a time; the lanes with
//                            the same target inside a step are found by OR-ing lane bits into a shared-memory
//                            word per target and ranked by lane, so the order stays stable; the lowest lane of
//                            a group hands the group's running position to the others by a shuffle (one warp
//                            barrier per step; the mask words of consecutive steps sit in alternating rows)
// 12 bytes of HBM traffic per entry (two reads of the table, one write of the positions).
#include "taot_internal.cuh"

namespace {

constexpr int kThreads = TAOT_STREAM_THREADS;
constexpr int kWarps = kThreads / 32;
constexpr int kWarpSpan = TAOT_CHUNK / kWarps;

struct DispatchArgs {
    const int32_t* idx;        // [L,T,k] rewritten routing table
    int32_t* dc;               // [L,R,NC,NB] chunk counts, then chunk bases
    const int32_t* tpos;       // [NB] sorted position of each bin
    const int32_t* torder;     // [NB] bin at each sorted position
    const int32_t* tdest;      // [NB] destination rank of each bin (R for the undeliverable bin)
    int32_t* send_counts;      // [L,R,R]
    int32_t* target_counts;    // [L,R,NB-1] or null
    int32_t* perm;             // [L,T,k]
    int32_t* info;
    int64_t layer_elems, seg;
    int32_t nc, R, NB, nbits;  // nbits: bits needed for a bin index in [0, NB)
};

__device__ __forceinline__ void chunk_span(const DispatchArgs& a, int64_t id, int64_t& goff, int32_t& len)
{
    const int32_t c = (int32_t)(id % a.nc);
    const int64_t lr = id / a.nc;
    const int64_t start = (int64_t)c * TAOT_CHUNK;
    len = (int32_t)((a.seg - start) < (int64_t)TAOT_CHUNK ? (a.seg - start) : (int64_t)TAOT_CHUNK);
    goff = (lr / a.R) * a.layer_elems + (lr % a.R) * a.seg + start;
}

__device__ __forceinline__ int bin_of(int32_t v, int NB) { return (unsigned)v < (unsigned)(NB - 1) ? v : NB - 1; }

__global__ void __launch_bounds__(kThreads)
dispatch_offsets_kernel(DispatchArgs a)
{
    extern __shared__ int32_t sh[];
    const int NB = a.NB, R = a.R, NC = a.nc;
    int32_t* tot = sh;                 // [NB] totals by bin
    int32_t* pref = tot + NB;          // [NB] exclusive prefix by bin, in destination order
    int32_t* sc = pref + NB;           // [R + 1] entries per destination rank (+ undeliverable)
    __shared__ int32_t wsum[kWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t lr = blockIdx.x;
    int32_t* dc = a.dc + lr * NC * (int64_t)NB;
    for (int r = tid; r <= R; r += kThreads) sc[r] = 0;
    for (int b = tid; b < NB; b += kThreads) {
        int32_t t = 0;
        for (int c = 0; c < NC; ++c) t += dc[(int64_t)c * NB + b];
        tot[b] = t;
    }
    __syncthreads();
    // exclusive scan of the totals taken in destination order: thread t owns sorted positions [t*per, (t+1)*per)
    const int per = (NB + kThreads - 1) / kThreads;
    const int p0 = tid * per, p1 = min(NB, p0 + per);
    int32_t local = 0;
    for (int p = p0; p < p1; ++p) local += tot[a.torder[p]];
    int32_t inc = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    int32_t run = inc - local;
    for (int w = 0; w < warp; ++w) run += wsum[w];
    for (int p = p0; p < p1; ++p) {
        const int b = a.torder[p];
        pref[b] = run;
        run += tot[b];
    }
    __syncthreads();
    for (int b = tid; b < NB; b += kThreads) {
        int32_t base = pref[b];
        for (int c = 0; c < NC; ++c) {
            const int32_t t = dc[(int64_t)c * NB + b];
            dc[(int64_t)c * NB + b] = base;
            base += t;
        }
        if (tot[b] != 0) atomicAdd(&sc[a.tdest[b]], tot[b]);
        if (a.target_counts && b < NB - 1) a.target_counts[lr * (int64_t)(NB - 1) + b] = tot[b];
    }
    __syncthreads();
    for (int r = tid; r < R; r += kThreads) a.send_counts[lr * R + r] = sc[r];
    if (tid == 0 && sc[R] != 0) atomicOr(a.info + (int32_t)(lr / R), TAOT_INFO_BAD_INDEX);
}

// ALT: the mask words of consecutive ranking steps sit in alternating rows (one warp barrier per step); otherwise one
// row and a second barrier per step, for target counts whose three rows would not fit in shared memory.
template <bool ALT>
__global__ void __launch_bounds__(kThreads)
dispatch_scatter_kernel(DispatchArgs a)
{
    extern __shared__ int32_t wh[];            // [kWarps][NB]: counts of the warp's span, then running positions;
                                               // then (ALT: 2 x) [kWarps][NB] lane masks of the steps being ranked
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NB = a.NB;
    const int64_t id = blockIdx.x;
    int64_t goff; int32_t len;
    chunk_span(a, id, goff, len);
    const int32_t* src = a.idx + goff;
    int32_t* dst = a.perm + goff;
    for (int q = tid; q < (ALT ? 3 : 2) * kWarps * NB; q += kThreads) wh[q] = 0;
    __syncthreads();
    const int s0 = warp * kWarpSpan, s1 = min(len, s0 + kWarpSpan);
    int32_t* mine = wh + warp * NB;
    unsigned* mask = reinterpret_cast<unsigned*>(wh + (kWarps + warp) * NB);
#pragma unroll 8
    for (int i = s0 + lane; i < s1; i += 32) atomicAdd(&mine[bin_of(__ldg(src + i), NB)], 1);
    __syncthreads();
    const int32_t* base = a.dc + id * (int64_t)NB;
    for (int b = tid; b < NB; b += kThreads) {
        int32_t run = base[b];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const int32_t t = wh[w * NB + b];
            wh[w * NB + b] = run;
            run += t;
        }
    }
    __syncthreads();
    const unsigned lt = (1u << lane) - 1u;
    constexpr int U = 4;
    unsigned* mask2 = ALT ? mask + kWarps * NB : mask;      // the second set of mask rows: steps alternate between the two
    for (int i0 = s0; i0 < s1; i0 += 32 * U) {
        int32_t v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u * 32 + lane;
            v[u] = i < s1 ? __ldg(src + i) : 0;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u * 32 + lane;
            const bool ok = i < s1;
            const int b = ok ? bin_of(v[u], NB) : 0;
            unsigned* mrow = (u & 1) ? mask2 : mask;
            // the lanes of this step that share my target: every lane ORs its bit into the target's word of the
            // warp's mask row (a set, so the result does not depend on the order of the atomics)
            if (ok) atomicOr(&mrow[b], 1u << lane);
            __syncwarp();
            const unsigned peers = ok ? mrow[b] : (1u << lane);
            // the lowest lane of a group reads the group's running position and hands it to the others by a shuffle,
            // which every lane reaches with its copy of the word read; only then does that lane move the position on
            // and clear the word.  The word is next written two steps later (the rows alternate) and the running
            // position is next read after the next step's barrier.
            const bool lead = ok && (peers & lt) == 0;
            int32_t first = lead ? mine[b] : 0;
            first = __shfl_sync(0xffffffffu, first, __ffs(peers) - 1);
            if (lead) {
                mine[b] = first + __popc(peers);
                mrow[b] = 0u;
            }
            if (ok) dst[i] = first + __popc(peers & lt);
            if (!ALT) __syncwarp();              // the cleared word is written again in the very next step
        }
    }
}

}  // namespace

int taot_launch_dispatch(taot_handle_t h, const int32_t* d_new_idx, int32_t* d_send_counts, int32_t* d_target_counts,
                         int32_t* d_perm, int32_t* d_info, void* ws, cudaStream_t st)
{
    const taot_params& p = h->p;
    DispatchArgs a;
    a.idx = d_new_idx;
    a.dc = reinterpret_cast<int32_t*>(static_cast<char*>(ws) + h->off_dc);
    a.tpos = h->d_tpos; a.torder = h->d_torder; a.tdest = h->d_tdest;
    a.send_counts = d_send_counts; a.target_counts = d_target_counts; a.perm = d_perm; a.info = d_info;
    a.layer_elems = p.T * p.k; a.seg = h->seg; a.nc = h->nc; a.R = p.R; a.NB = p.E + p.R * p.K + 1;
    const unsigned chunks = (unsigned)((int64_t)p.L * p.R * h->nc);
    a.nbits = 1;
    while ((1 << a.nbits) < a.NB) ++a.nbits;
    const size_t sm2 = sizeof(int32_t) * (2 * (size_t)a.NB + p.R + 1);
    const bool alt = sizeof(int32_t) * 3 * (size_t)kWarps * a.NB <= 64 * 1024;
    const size_t sm3 = sizeof(int32_t) * (alt ? 3 : 2) * (size_t)kWarps * a.NB;
    if (alt) TAOT_CUDA_OK(cudaFuncSetAttribute(dispatch_scatter_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3));
    else TAOT_CUDA_OK(cudaFuncSetAttribute(dispatch_scatter_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3));
    const int rc = taot_launch_chunk_counts(h, d_new_idx, a.dc, d_info, a.NB - 1, st);
    if (rc < 0) return rc;
    dispatch_offsets_kernel<<<(unsigned)((int64_t)p.L * p.R), kThreads, sm2, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    if (alt) dispatch_scatter_kernel<true><<<chunks, kThreads, sm3, st>>>(a);
    else dispatch_scatter_kernel<false><<<chunks, kThreads, sm3, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    return 3;
}
