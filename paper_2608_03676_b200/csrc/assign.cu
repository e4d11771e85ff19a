// Token reassignment: rewrite the routing table so that, within every (source rank, expert)
// group, the earliest entries move to the guest slots holding that expert (lowest slot first,
// X[r][s] entries each) and the rest stay.  ("Token routing is adjusted accordingly", Problem
// Formulation; the paper fixes the counts X, this rule fixes which entries.)
//
// One CTA per chunk of at most TAOT_CHUNK entries, the same chunks the histogram kernel counted.
// The chunk is loaded once into registers (64 entries per thread, all loads issued up front).
// From the per-chunk counts the CTA knows, for every expert, the ordinal range its entries
// occupy inside the (rank, expert) group; if that range falls inside one slot's quota (or
// outside all of them) the whole chunk maps that expert to one target and a shared-memory table
// lookup suffices.  Only experts whose range straddles a quota boundary need per-entry ordinals,
// which come from warp ballots over the register-resident chunk.  8 bytes of HBM traffic per
// entry: one read, one write.
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

__global__ void __launch_bounds__(kThreads)
assign_kernel(AssignArgs a)
{
    extern __shared__ int32_t sh[];
    const int E = a.E, S = a.R * a.K;
    int32_t* tab = sh;                  // [E]  >= 0: target for the whole chunk; -(1+b): boundary expert b
    int32_t* base = tab + E;            // [E]  ordinal of the chunk's first entry of e within (rank, e)
    int32_t* blist = base + E;          // [E]  boundary experts
    int32_t* cntw = blist + E;          // [E * kWarps] per-warp counts of each boundary expert
    int32_t* ent_s = cntw + E * kWarps; // [S]  slots this source rank feeds, ascending
    int32_t* ent_e = ent_s + S;         // [S]  their expert
    int32_t* ent_lo = ent_e + S;        // [S]  first ordinal the slot takes
    int32_t* ent_hi = ent_lo + S;       // [S]  one past the last
    __shared__ int s_wcnt[kWarps];
    __shared__ int s_nb;

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
    if (a.vec_ok) {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int32_t pos = wbase_elem + it * 128;
            if (pos + 3 < len) x[it] = ld_stream(reinterpret_cast<const int4*>(src + pos));
            else {
                x[it].x = pos < len ? src[pos] : -1;
                x[it].y = pos + 1 < len ? src[pos + 1] : -1;
                x[it].z = pos + 2 < len ? src[pos + 2] : -1;
                x[it].w = -1;
            }
        }
    } else {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int32_t pos = wbase_elem + it * 128;
            x[it].x = pos < len ? src[pos] : -1;
            x[it].y = pos + 1 < len ? src[pos + 1] : -1;
            x[it].z = pos + 2 < len ? src[pos + 2] : -1;
            x[it].w = pos + 3 < len ? src[pos + 3] : -1;
        }
    }

    // ---- slots fed by this source rank (X > 0), ascending slot order
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
    // ---- chunk-start ordinal and default target per expert
    const int32_t* ccseg = a.cc + lr * a.nc * (int64_t)E;
    for (int e = tid; e < E; e += kThreads) {
        int32_t b = 0;
        for (int cp = 0; cp < c; ++cp) b += ccseg[(int64_t)cp * E + e];
        base[e] = b;
        tab[e] = e;
    }
    if (tid == 0) s_nb = 0;
    // ordinal interval [lo, hi) each entry takes within its (rank, expert) group
    for (int q = tid; q < m; q += kThreads) {
        const int e = ent_e[q];
        int32_t lo = 0;
        for (int p = 0; p < q; ++p) lo += (ent_e[p] == e) ? ent_hi[p] : 0;
        ent_lo[q] = lo;
    }
    __syncthreads();
    for (int q = tid; q < m; q += kThreads) ent_hi[q] += ent_lo[q];
    __syncthreads();
    // classify: whole chunk range inside one interval -> table; straddling -> boundary expert
    for (int q = tid; q < m; q += kThreads) {
        const int e = ent_e[q];
        const int32_t cnt = ccseg[(int64_t)c * E + e];
        const int32_t b = base[e];
        if (cnt == 0 || ent_hi[q] <= b || ent_lo[q] >= b + cnt) continue;
        if (ent_lo[q] <= b && ent_hi[q] >= b + cnt) tab[e] = E + ent_s[q];
        else tab[e] = -1;
    }
    __syncthreads();
    for (int e = tid; e < E; e += kThreads)
        if (tab[e] == -1) {
            const int bi = atomicAdd(&s_nb, 1);
            blist[bi] = e;
            tab[e] = -(1 + bi);
        }
    __syncthreads();
    const int nb = s_nb;

    // ---- boundary experts: exact ordinals from ballots over the register-resident chunk
    unsigned long long done = 0ull;
    if (nb > 0) {
        for (int bi = 0; bi < nb; ++bi) {
            const int eb = blist[bi];
            int cnt = 0;
#pragma unroll
            for (int it = 0; it < kIters; ++it)
                cnt += (x[it].x == eb) + (x[it].y == eb) + (x[it].z == eb) + (x[it].w == eb);
            for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
            if (lane == 0) cntw[bi * kWarps + warp] = cnt;
        }
        __syncthreads();
        const unsigned lt = (1u << lane) - 1u;
        for (int bi = 0; bi < nb; ++bi) {
            const int eb = blist[bi];
            int32_t running = base[eb];
            for (int w = 0; w < warp; ++w) running += cntw[bi * kWarps + w];
            if (cntw[bi * kWarps + warp] == 0) continue;
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
                        int32_t target = eb;
                        for (int q = 0; q < m; ++q)
                            if (ent_e[q] == eb && ord >= ent_lo[q] && ord < ent_hi[q]) { target = E + ent_s[q]; break; }
                        xv[j] = target;
                        done |= 1ull << (it * 4 + j);
                        ++ord;
                    }
                }
                running += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
            }
        }
    }

    // ---- everything else: one table lookup per entry
    int bad = 0;
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
        int32_t* xv = reinterpret_cast<int32_t*>(&x[it]);
        const int32_t pos = wbase_elem + it * 128;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if ((done >> (it * 4 + j)) & 1ull) continue;
            const int32_t e = xv[j];
            if ((uint32_t)e < (uint32_t)E) xv[j] = tab[e];
            else if (pos + j < len) bad = 1;
        }
    }

    // ---- store
    if (a.vec_ok) {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int32_t pos = wbase_elem + it * 128;
            if (pos + 3 < len) st_stream(reinterpret_cast<int4*>(dst + pos), x[it]);
            else {
                if (pos < len) dst[pos] = x[it].x;
                if (pos + 1 < len) dst[pos + 1] = x[it].y;
                if (pos + 2 < len) dst[pos + 2] = x[it].z;
            }
        }
    } else {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            const int32_t pos = wbase_elem + it * 128;
            if (pos < len) dst[pos] = x[it].x;
            if (pos + 1 < len) dst[pos + 1] = x[it].y;
            if (pos + 2 < len) dst[pos + 2] = x[it].z;
            if (pos + 3 < len) dst[pos + 3] = x[it].w;
        }
    }
    bad = __syncthreads_or(bad);
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
    const size_t smem = sizeof(int32_t) * ((size_t)p.E * (3 + kWarps) + 4 * (size_t)S);
    TAOT_CUDA_OK(cudaFuncSetAttribute(assign_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t blocks = (int64_t)p.L * p.R * h->nc;
    assign_kernel<<<(unsigned)blocks, kThreads, smem, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
