// Token reassignment: rewrite the routing table so that, within every (source rank, expert)
// group, the earliest entries move to the guest slots holding that expert (lowest slot first,
// X[r][s] entries each) and the rest stay.  ("Token routing is adjusted accordingly", Problem
// Formulation; the paper fixes the counts X, this rule fixes which entries.)
//
// One CTA per chunk of at most TAOT_CHUNK entries, the same chunks the histogram kernel counted.
// The chunk is loaded once into registers (64 entries per thread, all loads issued up front);
// each warp owns 2048 contiguous entries.  The chunk counts of the histogram pass give the ordinal
// at which each expert's entries start in this chunk; a per-warp shared-memory histogram refines
// that to the start inside each warp's span.  If a warp's ordinal range for an expert falls inside
// one slot's quota (or outside all of them) every such entry of the warp has the same target and a
// per-warp lookup table suffices; only a (warp, expert) pair whose range straddles a quota boundary
// -- a handful per layer -- gets exact per-entry ordinals from warp ballots.  8 bytes of HBM traffic
// per entry: one read, one write.
#include "taot_internal.cuh"

namespace {

constexpr int kThreads = TAOT_STREAM_THREADS;
constexpr int kWarps = kThreads / 32;
constexpr int kIters = TAOT_CHUNK / (kThreads * 4);      // int4 loads per thread: 16
constexpr int kWarpSpan = TAOT_CHUNK / kWarps;           // entries one warp owns, contiguous: 2048

struct AssignArgs {
    const int32_t* topk;
    const int32_t* cc;
    const int32_t* slot_expert;
    const int32_t* X;
    int32_t* out;
    int32_t* info;
    int64_t layer_elems, seg;
    int32_t nc, R, E, K, vec_ok;
};

__device__ __forceinline__ int4 ld_stream(const int4* p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream(int4* p, const int4& v)
{
    asm volatile("st.global.cs.v4.s32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads)
assign_kernel(AssignArgs a)
{
    extern __shared__ int32_t sh[];
    const int E = a.E, S = a.R * a.K;
    int32_t* hw = sh;                   // [kWarps][E] per-warp histogram of the warp's 2048 entries
    int32_t* tabw = hw + kWarps * E;    // [kWarps][E] per-warp target table (-1: straddles a quota boundary)
    int32_t* base = tabw + kWarps * E;  // [E]  ordinal of the chunk's first entry of e within (rank, e)
    int32_t* ent_s = base + E;          // [S]  slots this source rank feeds, ascending
    int32_t* ent_e = ent_s + S;         // [S]  their expert
    int32_t* ent_lo = ent_e + S;        // [S]  first ordinal the slot takes
    int32_t* ent_hi = ent_lo + S;       // [S]  one past the last
    __shared__ int s_wcnt[kWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t id = blockIdx.x;
    const int32_t c = (int32_t)(id % a.nc);
    const int64_t lr = id / a.nc;
    const int32_t l = (int32_t)(lr / a.R);
    const int64_t start = (int64_t)c * TAOT_CHUNK;
    const int32_t len = (int32_t)((a.seg - start) < (int64_t)TAOT_CHUNK ? (a.seg - start) : (int64_t)TAOT_CHUNK);
    const int64_t goff = (int64_t)l * a.layer_elems + (lr % a.R) * a.seg + start;
    const int32_t* src = a.topk + goff;
    int32_t* dst = a.out + goff;

    // ---- the chunk, in registers; warp w owns entries [w*2048, w*2048+2048), 128 per iteration
    int4 x[kIters];
    const int32_t wbase_elem = warp * kWarpSpan + lane * 4;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int32_t pos = wbase_elem + it * 128;
        if (VEC && pos + 3 < len) x[it] = ld_stream(reinterpret_cast<const int4*>(src + pos));
        else {
            x[it].x = pos < len ? src[pos] : -1;
            x[it].y = pos + 1 < len ? src[pos + 1] : -1;
            x[it].z = pos + 2 < len ? src[pos + 2] : -1;
            x[it].w = pos + 3 < len ? src[pos + 3] : -1;
        }
    }

    // ---- while the loads fly: zero the histograms, chunk-start ordinals, the slots this rank feeds
    for (int i = tid; i < kWarps * E; i += kThreads) hw[i] = 0;
    const int32_t* ccseg = a.cc + lr * a.nc * (int64_t)E;
    for (int e = tid; e < E; e += kThreads) {
        int32_t b = 0;
        for (int cp = 0; cp < c; ++cp) b += ccseg[(int64_t)cp * E + e];
        base[e] = b;
    }
    const int32_t* Xrow = a.X + lr * S;
    const int32_t* se = a.slot_expert + (int64_t)l * S;
    int m = 0;
    for (int sb = 0; sb < S; sb += kThreads) {
        const int s = sb + tid;
        const int32_t xv = s < S ? Xrow[s] : 0;
        const int32_t ev = s < S ? se[s] : -1;
        const bool p = xv > 0 && ev >= 0 && ev < E;
        const unsigned bal = __ballot_sync(0xffffffffu, p);
        if (lane == 0) s_wcnt[warp] = __popc(bal);
        __syncthreads();
        int off = m;
        for (int w = 0; w < warp; ++w) off += s_wcnt[w];
        if (p) {
            const int q = off + __popc(bal & ((1u << lane) - 1u));
            ent_s[q] = s; ent_e[q] = ev; ent_hi[q] = xv;     // hi holds the count until the prefix below
        }
        for (int w = 0; w < kWarps; ++w) m += s_wcnt[w];
        __syncthreads();
    }
    // ordinal interval [lo, hi) each entry takes within its (rank, expert) group
    for (int q = tid; q < m; q += kThreads) {
        const int e = ent_e[q];
        int32_t lo = 0;
        for (int p = 0; p < q; ++p) lo += (ent_e[p] == e) ? ent_hi[p] : 0;
        ent_lo[q] = lo;
    }
    __syncthreads();
    for (int q = tid; q < m; q += kThreads) ent_hi[q] += ent_lo[q];

    // ---- per-warp histogram of the register-resident entries
    int32_t* myh = hw + warp * E;
    int bad = 0;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        const int32_t* xv = reinterpret_cast<const int32_t*>(&x[it]);
        const int32_t pos = wbase_elem + it * 128;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int32_t e = xv[j];
            if ((uint32_t)e < (uint32_t)E) atomicAdd(myh + e, 1);
            else if (pos + j < len) bad = 1;
        }
    }
    bad = __syncthreads_or(bad);          // also: every warp's histogram and ent_hi are complete

    // ---- this warp's table: default e; entries of this source rank override where they apply
    int32_t* myt = tabw + warp * E;
    for (int e = lane; e < E; e += 32) myt[e] = e;
    __syncwarp();
    for (int q = lane; q < m; q += 32) {
        const int e = ent_e[q];
        const int32_t cnt = myh[e];
        if (cnt == 0) continue;
        int32_t st = base[e];
        for (int w = 0; w < warp; ++w) st += hw[w * E + e];
        if (ent_hi[q] <= st || ent_lo[q] >= st + cnt) continue;
        myt[e] = (ent_lo[q] <= st && ent_hi[q] >= st + cnt) ? E + ent_s[q] : -1;   // at most one full cover
    }
    __syncwarp();

    // ---- (warp, expert) pairs that straddle a quota boundary: exact ordinals from ballots
    for (int eb0 = 0; eb0 < E; eb0 += 32) {
        const int ecand = eb0 + lane;
        unsigned todo = __ballot_sync(0xffffffffu, ecand < E && myt[ecand] == -1);
        while (todo) {
            const int eb = eb0 + __ffs(todo) - 1;
            todo &= todo - 1;
            int32_t running = base[eb];
            for (int w = 0; w < warp; ++w) running += hw[w * E + eb];
            const int32_t mine = myh[eb];
            int q0 = m, q1 = m;                  // entries of eb whose interval can touch [running, running+mine)
            for (int q = 0; q < m; ++q)
                if (ent_e[q] == eb && ent_hi[q] > running) { q0 = q; break; }
            for (int q = q0; q < m; ++q)
                if (ent_e[q] == eb && ent_lo[q] >= running + mine) { q1 = q; break; }
            const unsigned lt = (1u << lane) - 1u;
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                int32_t* xv = reinterpret_cast<int32_t*>(&x[it]);
                const bool m0 = xv[0] == eb, m1 = xv[1] == eb, m2 = xv[2] == eb, m3 = xv[3] == eb;
                const unsigned b0 = __ballot_sync(0xffffffffu, m0), b1 = __ballot_sync(0xffffffffu, m1);
                const unsigned b2 = __ballot_sync(0xffffffffu, m2), b3 = __ballot_sync(0xffffffffu, m3);
                if ((b0 | b1 | b2 | b3) == 0) continue;
                int32_t ord = running + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
                const bool mm[4] = {m0, m1, m2, m3};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (mm[j]) {
                        for (int q = q0; q < q1; ++q)
                            if (ent_e[q] == eb && ord >= ent_lo[q] && ord < ent_hi[q]) { xv[j] = E + ent_s[q]; break; }
                        ++ord;
                    }
                }
                running += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
            }
            // what is still eb in the registers stays eb; moved entries are now >= E and pass through
            if (lane == 0) myt[eb] = eb;
        }
        __syncwarp();
    }

    // ---- one table lookup per entry (values >= E or < 0 pass through unchanged), then store
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        int32_t* xv = reinterpret_cast<int32_t*>(&x[it]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int32_t e = xv[j];
            if ((uint32_t)e < (uint32_t)E) xv[j] = myt[e];
        }
        const int32_t pos = wbase_elem + it * 128;
        if (VEC && pos + 3 < len) st_stream(reinterpret_cast<int4*>(dst + pos), x[it]);
        else {
            if (pos < len) dst[pos] = x[it].x;
            if (pos + 1 < len) dst[pos + 1] = x[it].y;
            if (pos + 2 < len) dst[pos + 2] = x[it].z;
            if (pos + 3 < len) dst[pos + 3] = x[it].w;
        }
    }
    if (bad && tid == 0) atomicOr(a.info + l, TAOT_INFO_BAD_INDEX);
}

}  // namespace

int taot_launch_assign(taot_handle_t h, const int32_t* d_topk, const int32_t* d_cc,
                       const int32_t* d_slot_expert, const int32_t* d_X, int32_t* d_new_idx,
                       int32_t* d_info, cudaStream_t st)
{
    const taot_params& p = h->p;
    AssignArgs a;
    a.topk = d_topk; a.cc = d_cc; a.slot_expert = d_slot_expert; a.X = d_X; a.out = d_new_idx; a.info = d_info;
    a.layer_elems = p.T * p.k; a.seg = h->seg; a.nc = h->nc; a.R = p.R; a.E = p.E; a.K = p.K;
    a.vec_ok = ((reinterpret_cast<uintptr_t>(d_topk) & 15) == 0) &&
               ((reinterpret_cast<uintptr_t>(d_new_idx) & 15) == 0) && (h->seg % 4 == 0);
    const int S = p.R * p.K;
    const size_t smem = sizeof(int32_t) * ((size_t)p.E * (2 * kWarps + 1) + 4 * (size_t)S);
    const int64_t blocks = (int64_t)p.L * p.R * h->nc;
    if (a.vec_ok) {
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        assign_kernel<true><<<(unsigned)blocks, kThreads, smem, st>>>(a);
    } else {
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        assign_kernel<false><<<(unsigned)blocks, kThreads, smem, st>>>(a);
    }
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
