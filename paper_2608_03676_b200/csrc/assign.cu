// Token reassignment: rewrite the routing table so that, within every (source rank, expert)
// group, the earliest entries move to the guest slots holding that expert (lowest slot first,
// X[r][s] entries each) and the rest stay.  ("Token routing is adjusted accordingly", Problem
// Formulation; the paper fixes the counts X, this rule fixes which entries.)
//
// One CTA per chunk of at most TAOT_CHUNK entries, the same chunks the histogram kernel counted.
// The chunk is loaded once into registers (64 entries per thread, all loads issued up front);
// each warp owns 2048 contiguous entries.  The chunk counts of the histogram pass give, for every
// expert, the ordinal range its entries occupy in this chunk.  If that range falls inside one
// slot's quota (or outside all of them) every such entry of the chunk has the same target: one
// shared-memory table lookup per entry, and that is all most chunks need.  An expert whose range
// straddles a quota boundary (about one chunk in five has one) is counted per warp from the
// registers; warps that do not contain the boundary still get a single target for it, and only the
// one warp that does computes exact per-entry ordinals from ballots.  The per-chunk tables are built
// by a small kernel with one CTA per (layer, source rank) segment, so that the streaming kernel's
// common path is: 16 loads in flight, one table row from L2, 64 lookups, 16 stores.  8 bytes of HBM
// traffic per entry: one read, one write.  Out-of-range indices are copied through (the histogram pass, whose
// counts this kernel consumes, is the one that flags them).
#include <cstdio>

#include "taot_internal.cuh"

namespace {

constexpr int kThreads = TAOT_STREAM_THREADS;
constexpr int kWarps = kThreads / 32;
constexpr int kIters = TAOT_CHUNK / (kThreads * 4);      // int4 loads per thread: 16
constexpr int kWarpSpan = TAOT_CHUNK / kWarps;           // entries one warp owns, contiguous: 2048

struct AssignArgs {
    const int32_t* topk;
    const int32_t* cc;
    int32_t* tabg;          // [L,R,NC,E] per-chunk target tables written by the prep kernel
    int32_t* nbg;           // [L,R,NC]   number of boundary experts of each chunk
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

// Shared by both kernels: the slots this source rank feeds (X > 0), ascending, with the ordinal
// interval [lo, hi) each takes inside its (rank, expert) group.  Returns the number of entries.
// On return ent_hi holds COUNTS (hi - lo); the caller adds ent_lo after its last use of the counts.
__device__ int build_entries(const int32_t* Xrow, const int32_t* se, int S, int E, int32_t* ent_s,
                             int32_t* ent_e, int32_t* ent_lo, int32_t* ent_hi, int* s_wcnt)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NT = blockDim.x, NWB = NT >> 5;
    int m = 0;
    for (int sb = 0; sb < S; sb += NT) {
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
            ent_s[q] = s; ent_e[q] = ev; ent_hi[q] = xv;
        }
        for (int w = 0; w < NWB; ++w) m += s_wcnt[w];
        __syncthreads();
    }
    for (int q = tid; q < m; q += NT) {
        const int e = ent_e[q];
        int32_t lo = 0;
        for (int p = 0; p < q; ++p) lo += (ent_e[p] == e) ? ent_hi[p] : 0;
        ent_lo[q] = lo;
    }
    __syncthreads();
    return m;
}

// One CTA per (layer, source rank): the target table of every chunk of the segment.
// tab[e] = e (stays), E + s (the chunk's whole ordinal range of e lies in slot s's quota) or -1
// (the range straddles a quota boundary: a boundary expert of that chunk).
__global__ void __launch_bounds__(kThreads)
assign_prep_kernel(AssignArgs a)
{
    extern __shared__ int32_t sh[];
    const int E = a.E, S = a.R * a.K;
    int32_t* tab = sh;                  // [E]
    int32_t* base = tab + E;            // [E] running ordinal at the start of the current chunk
    int32_t* ent_s = base + E;          // [S]
    int32_t* ent_e = ent_s + S;
    int32_t* ent_lo = ent_e + S;
    int32_t* ent_hi = ent_lo + S;
    __shared__ int s_wcnt[kWarps];
    __shared__ int s_nb;
    const int tid = threadIdx.x;
    const int64_t lr = blockIdx.x;
    const int32_t l = (int32_t)(lr / a.R);
    const int m = build_entries(a.X + lr * S, a.slot_expert + (int64_t)l * S, S, E, ent_s, ent_e, ent_lo, ent_hi, s_wcnt);
    for (int e = tid; e < E; e += kThreads) base[e] = 0;
    const int32_t* ccseg = a.cc + lr * a.nc * (int64_t)E;
    for (int c = 0; c < a.nc; ++c) {
        for (int e = tid; e < E; e += kThreads) tab[e] = e;
        if (tid == 0) s_nb = 0;
        __syncthreads();
        for (int q = tid; q < m; q += kThreads) {
            const int e = ent_e[q];
            const int32_t lo = ent_lo[q], hi = lo + ent_hi[q];
            const int32_t cnt = ccseg[(int64_t)c * E + e];
            const int32_t b = base[e];
            if (!(cnt == 0 || hi <= b || lo >= b + cnt))
                tab[e] = (lo <= b && hi >= b + cnt) ? E + ent_s[q] : -1;      // at most one full cover per expert
        }
        __syncthreads();
        int32_t* out = a.tabg + (lr * a.nc + c) * (int64_t)E;
        for (int e = tid; e < E; e += kThreads) {
            const int32_t t = tab[e];
            out[e] = t;
            if (t == -1) atomicAdd(&s_nb, 1);
            base[e] += ccseg[(int64_t)c * E + e];
        }
        __syncthreads();
        if (tid == 0) a.nbg[lr * a.nc + c] = s_nb;
        __syncthreads();
    }
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads, 2)
assign_kernel(AssignArgs a)
{
    extern __shared__ int32_t sh[];
    const int E = a.E, S = a.R * a.K;
    int32_t* tab = sh;                  // [E]  >= 0: target for the whole chunk; -(1+b): boundary expert b
    int32_t* base = tab + E;            // [E]  ordinal of the chunk's first entry of e within (rank, e)
    int32_t* blist = base + E;          // [E]  boundary experts of this chunk
    int32_t* cntw = blist + E;          // [E * kWarps] per-warp counts of each boundary expert
    int32_t* wtab = cntw + E * kWarps;  // [kWarps][E] per-warp tables, used only if the chunk has a boundary expert
    int32_t* ent_s = wtab + E * kWarps; // [S]  slots this source rank feeds, ascending
    int32_t* ent_e = ent_s + S;         // [S]  their expert
    int32_t* ent_lo = ent_e + S;        // [S]  first ordinal the slot takes
    int32_t* ent_hi = ent_lo + S;       // [S]  one past the last
    __shared__ int s_wcnt[kWarps];
    __shared__ int s_nb;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t id = blockIdx.x;
    const int nb = a.nbg[id];
    const int32_t c = (int32_t)(id % a.nc);
    const int64_t lr = id / a.nc;
    const int32_t l = (int32_t)(lr / a.R);
    const int64_t start = (int64_t)c * TAOT_CHUNK;
    const int32_t len = (int32_t)((a.seg - start) < (int64_t)TAOT_CHUNK ? (a.seg - start) : (int64_t)TAOT_CHUNK);
    const int64_t goff = (int64_t)l * a.layer_elems + (lr % a.R) * a.seg + start;
    const int32_t* src = a.topk + goff;
    int32_t* dst = a.out + goff;
    const bool full = VEC && (len == TAOT_CHUNK);

    // ---- the chunk, in registers; warp w owns entries [w*2048, w*2048+2048), 128 per iteration
    int4 x[kIters];
    const int32_t wbase_elem = warp * kWarpSpan + lane * 4;
    if (full) {
#pragma unroll
        for (int it = 0; it < kIters; ++it)
            x[it] = ld_stream(reinterpret_cast<const int4*>(src + wbase_elem + it * 128));
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

    // ---- this chunk's table row (built by the prep kernel) and its boundary count
    const int32_t* trow = a.tabg + id * (int64_t)E;
    for (int e = tid; e < E; e += kThreads) tab[e] = trow[e];
    __syncthreads();
    const int32_t* lut = tab;

    if (nb > 0) {
        // ---- rare path: rebuild this rank's quota intervals, refine the boundary experts per warp
        const int m = build_entries(a.X + lr * S, a.slot_expert + (int64_t)l * S, S, E, ent_s, ent_e, ent_lo, ent_hi, s_wcnt);
        for (int q = tid; q < m; q += kThreads) ent_hi[q] += ent_lo[q];
        const int32_t* ccseg = a.cc + lr * a.nc * (int64_t)E;
        if (tid == 0) s_nb = 0;
        __syncthreads();
        for (int e = tid; e < E; e += kThreads)
            if (tab[e] == -1) {
                int32_t b = 0;
                for (int cp = 0; cp < c; ++cp) b += ccseg[(int64_t)cp * E + e];
                const int bi = atomicAdd(&s_nb, 1);
                blist[bi] = e;
                base[bi] = b;
                tab[e] = e;                              // refined per warp below
            }
        __syncthreads();
        // per-warp counts of the boundary experts, from the registers
        for (int bi = 0; bi < nb; ++bi) {
            const int eb = blist[bi];
            int cnt = 0;
#pragma unroll
            for (int it = 0; it < kIters; ++it)
                cnt += (x[it].x == eb) + (x[it].y == eb) + (x[it].z == eb) + (x[it].w == eb);
            for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
            if (lane == 0) cntw[bi * kWarps + warp] = cnt;
        }
        int32_t* myt = wtab + warp * E;
        for (int e = lane; e < E; e += 32) myt[e] = tab[e];
        __syncthreads();
        const unsigned lt = (1u << lane) - 1u;
        for (int bi = 0; bi < nb; ++bi) {
            const int eb = blist[bi];
            const int32_t mine = cntw[bi * kWarps + warp];
            int32_t running = base[bi];
            for (int w = 0; w < warp; ++w) running += cntw[bi * kWarps + w];
            // this warp's ordinals of eb are [running, running + mine): inside one interval, outside all, or straddling
            int32_t target = eb;
            bool straddle = false;
            int q0 = m, q1 = m;
            for (int q = 0; q < m; ++q) {
                if (ent_e[q] != eb || mine == 0) continue;
                if (ent_hi[q] <= running || ent_lo[q] >= running + mine) continue;
                if (ent_lo[q] <= running && ent_hi[q] >= running + mine) target = E + ent_s[q];
                else { straddle = true; if (q0 == m) q0 = q; q1 = q + 1; }
            }
            if (!straddle) {
                if (lane == 0) myt[eb] = target;
                continue;
            }
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
        }
        __syncwarp();
        lut = myt;
    }

    // ---- one table lookup per entry (values >= E or < 0 pass through unchanged), then store
    if (full) {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            int32_t* xv = reinterpret_cast<int32_t*>(&x[it]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int32_t e = xv[j];
                if ((uint32_t)e < (uint32_t)E) xv[j] = lut[e];
            }
            st_stream(reinterpret_cast<int4*>(dst + wbase_elem + it * 128), x[it]);
        }
    } else {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
            int32_t* xv = reinterpret_cast<int32_t*>(&x[it]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int32_t e = xv[j];
                if ((uint32_t)e < (uint32_t)E) xv[j] = lut[e];
            }
            const int32_t pos = wbase_elem + it * 128;
            if (pos < len) dst[pos] = x[it].x;
            if (pos + 1 < len) dst[pos + 1] = x[it].y;
            if (pos + 2 < len) dst[pos + 2] = x[it].z;
            if (pos + 3 < len) dst[pos + 3] = x[it].w;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Persistent, bulk-copy-pipelined version of the rewrite (used when the routing table is 16-byte
// aligned and E is a multiple of 4).  One CTA per SM walks chunks blockIdx.x, +gridDim.x, ...; a
// single thread keeps kStages-1 chunks in flight with cp.async.bulk (global -> shared, completion
// counted on an mbarrier per stage, no multicast), so the loads of the next chunks overlap the
// lookups and stores of the current one.  Each stage carries the chunk (<= 64 KB) and its table row.
// Arithmetic and rare path are those of assign_kernel; the chunk is read from shared memory
// instead of registers.

constexpr int kSThreads = 256;
constexpr int kSWarps = kSThreads / 32;
constexpr int kSWarpSpan = TAOT_CHUNK / kSWarps;        // 2048 entries per warp, contiguous
constexpr int kSIters = kSWarpSpan / 128;               // 16 x 16-byte accesses per lane
constexpr uint32_t kBulkPiece = 8192;                   // bytes per bulk copy: several pieces in flight per chunk
constexpr uint32_t kWaitSpins = 1u << 20;               // bound on mbarrier polling (each poll can itself block for a while)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Poll until the phase with the given parity completes; false if the spin bound ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity)
{
    const uint32_t addr = smem_u32(bar);
    for (uint32_t spin = 0; spin < kWaitSpins; ++spin) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

struct StreamLayout {
    int stages;
    size_t off_tab, off_scratch, bytes;       // chunk buffers start at 0
};

StreamLayout stream_layout(int E, int S)
{
    const size_t scratch = sizeof(int32_t) * ((size_t)E * (2 + 2 * kSWarps) + 4 * (size_t)S);   // base, blist, cntw, wtab, ent_*
    StreamLayout L;
    const size_t per_stage = (size_t)TAOT_CHUNK * 4 + (size_t)E * 4;
    const size_t budget = 220 * 1024;
    int st = (int)((budget - scratch - 256) / per_stage);
    L.stages = st > 4 ? 4 : st;
    L.off_tab = (size_t)L.stages * TAOT_CHUNK * 4;
    L.off_scratch = L.off_tab + (size_t)L.stages * E * 4;
    L.bytes = L.off_scratch + scratch;
    return L;
}

__global__ void __launch_bounds__(kSThreads, 1)
assign_stream_kernel(AssignArgs a, int stages, uint32_t off_tab, uint32_t off_scratch, int64_t nchunks)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bars[4];
    __shared__ int s_wcnt[32];
    __shared__ int s_nb;
    const int E = a.E, S = a.R * a.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* scratch = reinterpret_cast<int32_t*>(smem + off_scratch);
    int32_t* base = scratch;                    // [E]  start ordinal of each boundary expert (indexed by its list position)
    int32_t* blist = base + E;                  // [E]
    int32_t* cntw = blist + E;                  // [E * kSWarps]
    int32_t* wtab = cntw + E * kSWarps;         // [kSWarps][E]
    int32_t* ent_s = wtab + E * kSWarps;        // [S] ...
    int32_t* ent_e = ent_s + S;
    int32_t* ent_lo = ent_e + S;
    int32_t* ent_hi = ent_lo + S;

    if (tid == 0) {
        for (int st = 0; st < stages; ++st) mbar_init(&bars[st], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto chunk_geometry = [&](int64_t id, int64_t& goff, int32_t& len) {
        const int32_t c = (int32_t)(id % a.nc);
        const int64_t lr = id / a.nc;
        const int64_t start = (int64_t)c * TAOT_CHUNK;
        len = (int32_t)((a.seg - start) < (int64_t)TAOT_CHUNK ? (a.seg - start) : (int64_t)TAOT_CHUNK);
        goff = (lr / a.R) * a.layer_elems + (lr % a.R) * a.seg + start;
    };
    auto issue = [&](int64_t id, int st) {      // one thread: arm the stage and start its two copies
        int64_t goff; int32_t len;
        chunk_geometry(id, goff, len);
        const uint32_t bytes = (uint32_t)len * 4u;
        mbar_expect_tx(&bars[st], bytes + (uint32_t)E * 4u);
        unsigned char* dstb = smem + (size_t)st * TAOT_CHUNK * 4;
        const unsigned char* srcb = reinterpret_cast<const unsigned char*>(a.topk + goff);
        for (uint32_t o = 0; o < bytes; o += kBulkPiece)
            bulk_load(dstb + o, srcb + o, (bytes - o) < kBulkPiece ? (bytes - o) : kBulkPiece, &bars[st]);
        bulk_load(smem + off_tab + (size_t)st * E * 4, a.tabg + id * (int64_t)E, (uint32_t)E * 4u, &bars[st]);
    };

    const int64_t first = blockIdx.x, stride = gridDim.x;
    if (tid == 0)
        for (int st = 0; st < stages; ++st)
            if (first + st * stride < nchunks) issue(first + st * stride, st);

    int64_t it_global = 0;
    for (int64_t id = first; id < nchunks; id += stride, ++it_global) {
        const int st = (int)(it_global % stages);
        const uint32_t parity = (uint32_t)((it_global / stages) & 1);
        const int nb = a.nbg[id];
        int64_t goff; int32_t len;
        chunk_geometry(id, goff, len);
        const int64_t lr = id / a.nc;
        const int32_t c = (int32_t)(id % a.nc);
        const int32_t l = (int32_t)(lr / a.R);
        int32_t* buf = reinterpret_cast<int32_t*>(smem + (size_t)st * TAOT_CHUNK * 4);
        const int32_t* tab = reinterpret_cast<const int32_t*>(smem + off_tab + (size_t)st * E * 4);
        int32_t* dst = a.out + goff;

        const bool ok = mbar_wait(&bars[st], parity);
        if (__syncthreads_or(!ok)) {
            // the copy never completed: report, give the copies still in flight one more bounded chance to land
            // (their destination is this CTA's shared memory), and leave
            if (tid == 0) {
                atomicOr(a.info + l, TAOT_INFO_INTERNAL);
                for (int s2 = 0; s2 < stages; ++s2) {
                    const int64_t use = (it_global + ((s2 - st + stages) % stages)) / stages;
                    (void)mbar_wait(&bars[s2], (uint32_t)(use & 1));
                }
            }
            __syncthreads();
            return;
        }
        const int32_t wbase = warp * kSWarpSpan + lane * 4;
        const int32_t* lut = tab;
        if (nb > 0) {
            // ---- rare path: this rank's quota intervals, per-warp refinement of the boundary experts
            const int m = build_entries(a.X + lr * S, a.slot_expert + (int64_t)l * S, S, E, ent_s, ent_e, ent_lo, ent_hi, s_wcnt);
            for (int q = tid; q < m; q += kSThreads) ent_hi[q] += ent_lo[q];
            const int32_t* ccseg = a.cc + lr * a.nc * (int64_t)E;
            if (tid == 0) s_nb = 0;
            __syncthreads();
            for (int e = tid; e < E; e += kSThreads)
                if (tab[e] == -1) {
                    int32_t b = 0;
                    for (int cp = 0; cp < c; ++cp) b += ccseg[(int64_t)cp * E + e];
                    const int bi = atomicAdd(&s_nb, 1);
                    blist[bi] = e;
                    base[bi] = b;
                }
            __syncthreads();
#pragma unroll 1
            for (int bi = 0; bi < nb; ++bi) {
                const int eb = blist[bi];
                int cnt = 0;
#pragma unroll 4
                for (int it = 0; it < kSIters; ++it) {
                    const int32_t pos = wbase + it * 128;
                    if (pos < len) {
                        const int4 v = *reinterpret_cast<const int4*>(buf + pos);
                        cnt += (v.x == eb) + (v.y == eb) + (v.z == eb) + (v.w == eb);
                    }
                }
                for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
                if (lane == 0) cntw[bi * kSWarps + warp] = cnt;
            }
            int32_t* myt = wtab + warp * E;
            for (int e = lane; e < E; e += 32) { const int32_t t = tab[e]; myt[e] = t == -1 ? e : t; }
            __syncthreads();
            const unsigned lt = (1u << lane) - 1u;
#pragma unroll 1
            for (int bi = 0; bi < nb; ++bi) {
                const int eb = blist[bi];
                const int32_t mine = cntw[bi * kSWarps + warp];
                int32_t running = base[bi];
                for (int w = 0; w < warp; ++w) running += cntw[bi * kSWarps + w];
                // this warp's ordinals of eb are [running, running + mine): inside one interval, outside all, or
                // straddling; the (at most two, else a list walk) intervals it straddles are kept in registers
                int32_t target = eb;
                int nstr = 0, q0 = m, q1 = m;
                int32_t lo0 = 0, hi0 = 0, t0 = eb, lo1 = 0, hi1 = 0, t1 = eb;
                for (int q = 0; q < m; ++q) {
                    if (ent_e[q] != eb || mine == 0) continue;
                    if (ent_hi[q] <= running || ent_lo[q] >= running + mine) continue;
                    if (ent_lo[q] <= running && ent_hi[q] >= running + mine) { target = E + ent_s[q]; continue; }
                    if (nstr == 0) { lo0 = ent_lo[q]; hi0 = ent_hi[q]; t0 = E + ent_s[q]; q0 = q; }
                    else if (nstr == 1) { lo1 = ent_lo[q]; hi1 = ent_hi[q]; t1 = E + ent_s[q]; }
                    ++nstr;
                    q1 = q + 1;
                }
                if (nstr == 0) {
                    if (lane == 0) myt[eb] = target;
                    continue;
                }
#pragma unroll 1
                for (int it = 0; it < kSIters; ++it) {           // kept rolled: this code runs rarely and must stay small
                    const int32_t pos = wbase + it * 128;
                    int4 v = make_int4(-1, -1, -1, -1);
                    if (pos < len) v = *reinterpret_cast<const int4*>(buf + pos);
                    int32_t* xv = reinterpret_cast<int32_t*>(&v);
                    const bool m0 = xv[0] == eb, m1 = xv[1] == eb, m2 = xv[2] == eb, m3 = xv[3] == eb;
                    const unsigned b0 = __ballot_sync(0xffffffffu, m0), b1 = __ballot_sync(0xffffffffu, m1);
                    const unsigned b2 = __ballot_sync(0xffffffffu, m2), b3 = __ballot_sync(0xffffffffu, m3);
                    if ((b0 | b1 | b2 | b3) == 0) continue;
                    int32_t ord = running + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
                    const bool mm[4] = {m0, m1, m2, m3};
                    bool changed = false;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (mm[j]) {
                            if (nstr <= 2) {
                                if (ord >= lo0 && ord < hi0) { xv[j] = t0; changed = true; }
                                else if (nstr == 2 && ord >= lo1 && ord < hi1) { xv[j] = t1; changed = true; }
                            } else {
                                for (int q = q0; q < q1; ++q)
                                    if (ent_e[q] == eb && ord >= ent_lo[q] && ord < ent_hi[q]) { xv[j] = E + ent_s[q]; changed = true; break; }
                            }
                            ++ord;
                        }
                    }
                    if (changed) *reinterpret_cast<int4*>(buf + pos) = v;        // moved entries are now >= E and pass through
                    running += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
                }
            }
            __syncwarp();
            lut = myt;
        }
        // ---- one table lookup per entry (values >= E or < 0 pass through unchanged), then store
#pragma unroll 4
        for (int it = 0; it < kSIters; ++it) {
            const int32_t pos = wbase + it * 128;
            if (pos < len) {
                int4 v = *reinterpret_cast<const int4*>(buf + pos);
#ifndef TAOT_DBG_NOLOOKUP
                if ((uint32_t)v.x < (uint32_t)E) v.x = lut[v.x];
                if ((uint32_t)v.y < (uint32_t)E) v.y = lut[v.y];
                if ((uint32_t)v.z < (uint32_t)E) v.z = lut[v.z];
                if ((uint32_t)v.w < (uint32_t)E) v.w = lut[v.w];
#endif
#ifdef TAOT_DBG_NOSTORE
                if (v.x == 0x7fffffff)
#endif
                st_stream(reinterpret_cast<int4*>(dst + pos), v);
            }
        }
        __syncthreads();                         // everyone is done with this stage's buffers
        if (tid == 0 && id + (int64_t)stages * stride < nchunks) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(id + (int64_t)stages * stride, st);
        }
    }
}

}  // namespace

int taot_launch_assign(taot_handle_t h, const int32_t* d_topk, const int32_t* d_cc, int32_t* d_tabg,
                       int32_t* d_nbg, const int32_t* d_slot_expert, const int32_t* d_X, int32_t* d_new_idx,
                       int32_t* d_info, cudaStream_t st)
{
    const taot_params& p = h->p;
    AssignArgs a;
    a.topk = d_topk; a.cc = d_cc; a.tabg = d_tabg; a.nbg = d_nbg;
    a.slot_expert = d_slot_expert; a.X = d_X; a.out = d_new_idx; a.info = d_info;
    a.layer_elems = p.T * p.k; a.seg = h->seg; a.nc = h->nc; a.R = p.R; a.E = p.E; a.K = p.K;
    a.vec_ok = ((reinterpret_cast<uintptr_t>(d_topk) & 15) == 0) &&
               ((reinterpret_cast<uintptr_t>(d_new_idx) & 15) == 0) && (h->seg % 4 == 0);
    const int S = p.R * p.K;
    const size_t smem_prep = sizeof(int32_t) * (2 * (size_t)p.E + 4 * (size_t)S);
    assign_prep_kernel<<<(unsigned)((int64_t)p.L * p.R), kThreads, smem_prep, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    const size_t smem = sizeof(int32_t) * ((size_t)p.E * (3 + 2 * kWarps) + 4 * (size_t)S);
    const unsigned blocks = (unsigned)((int64_t)p.L * p.R * h->nc);
    const StreamLayout sl = stream_layout(p.E, S);
    if (a.vec_ok && p.E % 4 == 0 && sl.stages >= 2) {
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sl.bytes));
        const unsigned grid = blocks < (unsigned)h->sm_count ? blocks : (unsigned)h->sm_count;
        assign_stream_kernel<<<grid, kSThreads, sl.bytes, st>>>(a, sl.stages, (uint32_t)sl.off_tab, (uint32_t)sl.off_scratch,
                                                              (int64_t)blocks);
    } else if (a.vec_ok) {
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        assign_kernel<true><<<blocks, kThreads, smem, st>>>(a);
    } else {
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        assign_kernel<false><<<blocks, kThreads, smem, st>>>(a);
    }
    TAOT_CUDA_OK(cudaGetLastError());
    return 2;
}
