// Token reassignment: rewrite the routing table so that, within every (source rank, expert)
// group, the earliest entries move to the guest slots holding that expert (lowest slot first,
// X[r][s] entries each) and the rest stay.  (Problem Formulation: the paper fixes the counts X
// and leaves the per-token rule open; this rule fixes which entries move.)
//
// Within a (rank, expert) group the slots take consecutive ordinal intervals [0,x1), [x1,x1+x2), ...
// The chunk counts of the histogram pass say which ordinals of each expert fall into each chunk of
// at most TAOT_CHUNK entries, so for most (chunk, expert) pairs every entry has the same target and
// the rewrite is a table lookup.  Where an interval ends strictly inside a chunk's ordinal range
// (a "split": at most one per slot this rank feeds; one chunk in five to two in five has one), the entries
// before the split position go to that slot and the later ones follow the next interval.  One kernel:
//   assign_chunk_kernel  one CTA per chunk, every chunk in one sweep over the table.  The chunk is staged in shared
//                        memory with bulk asynchronous copies (cp.async.bulk + mbarrier, no multicast, an L2
//                        evict-first policy: the table is read once); while they are in flight the CTA builds the
//                        chunk's table expert -> target (of the chunk's LAST entry of that expert) and its split
//                        records (expert, in-chunk ordinal, slot before) from X, the slots' experts and the chunk
//                        counts; three CTAs per SM keep copies, lookups and 16-byte streaming stores of different
//                        chunks in flight.  A chunk without a split is one table lookup per entry; a chunk with
//                        splits is read three times from shared memory --
//                        per-warp counts of the split experts, ballots in the one warp that holds a split to find
//                        its flat position, then the rewrite with "expert e before position P -> slot" as
//                        predicated overrides.  A routing table that is not 16-byte aligned or whose segments are
//                        not multiples of 4 entries takes the same kernel without staging, with ordinary loads.
// One sweep over all chunks matters: two kernels that each took part of the chunks (a persistent pipeline for the
// chunks without a split, a per-chunk kernel for the rest) were measured at 5.4-5.7 TB/s on their parts, a single
// sweep at 6.3-6.5 TB/s -- the memory system serves a contiguous sweep better than two interleaved subsets.
// 8 bytes of HBM traffic per entry (one read, one write) -- or 5 where the histogram pass has left the table as one byte
// per entry beside its counts (at most 256 experts, 16-byte aligned tables, segments of a multiple of 16 entries): the
// rewrite only needs to know each entry's expert, so it stages those 16 KB per chunk instead of 64 KB of the table; a chunk
// that holds a value which is no expert (flagged by the histogram pass) is read from the table itself.  Out-of-range
// indices are copied through (the histogram pass, whose counts this path consumes, is the one that flags them).
#include <type_traits>
#include "taot_internal.cuh"

namespace {

constexpr int kThreads = TAOT_STREAM_THREADS;
constexpr int kWarps = kThreads / 32;
constexpr int kWarpSpan = TAOT_CHUNK / kWarps;           // entries one warp owns, contiguous: 2048
constexpr int kIters = kWarpSpan / 128;                  // 16-byte accesses per lane: 16
constexpr int kFewSplits = 4;                            // splits of a chunk that are applied as predicated overrides from registers

struct AssignArgs {
    const int32_t* topk;
    const int32_t* cc;          // [L,R,NC,E] chunk counts (histogram pass)
    const int32_t* slot_expert;
    const int32_t* X;
    int32_t* out;
    int32_t* info;
    const uint8_t* tb;          // the table as one byte per entry (histogram pass), or null
    const int32_t* tbflag;      // [L,R,NC] nonzero: the chunk holds a value that is no expert (its bytes are not used)
    int64_t layer_elems, seg;
    int32_t nc, R, E, K;
};

__device__ __forceinline__ void st_stream(int4* p, const int4& v)
{
    asm volatile("st.global.cs.v4.s32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ void chunk_geometry(const AssignArgs& a, int64_t id, int64_t& goff, int32_t& len)
{
    const int32_t c = (int32_t)(id % a.nc);
    const int64_t lr = id / a.nc;
    const int64_t start = (int64_t)c * TAOT_CHUNK;
    len = (int32_t)((a.seg - start) < (int64_t)TAOT_CHUNK ? (a.seg - start) : (int64_t)TAOT_CHUNK);
    goff = (lr / a.R) * a.layer_elems + (lr % a.R) * a.seg + start;
}

// The slots this source rank feeds (X > 0), ascending, with the ordinal interval [lo, hi) each takes
// inside its (rank, expert) group.  Returns the number of entries.
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
            ent_s[q] = s; ent_e[q] = ev; ent_hi[q] = xv;         // count for now
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
    for (int q = tid; q < m; q += NT) ent_hi[q] += ent_lo[q];
    __syncthreads();
    return m;
}

// Flat position, inside the chunk held at `buf`, of the entry of expert eb whose in-chunk ordinal is rel
// (entries of eb before it belong to the slot whose quota ends there).  Block-wide: warp w owns entries
// [w*2048, (w+1)*2048); per-warp counts, then ballots in the one warp that holds the entry.
// four entries at pos (a multiple of 4) of a chunk held as one byte per entry
__device__ __forceinline__ int4 unpack_bytes(const void* buf, int32_t pos)
{
    const uint32_t w = *reinterpret_cast<const uint32_t*>(static_cast<const uint8_t*>(buf) + pos);
    return make_int4((int)(w & 255u), (int)((w >> 8) & 255u), (int)((w >> 16) & 255u), (int)(w >> 24));
}

template <bool VEC, bool BYTES>
__device__ int32_t locate_split(const void* bufv, int32_t len, int eb, int rel, int* s_cntw, int* s_pos)
{
    const int32_t* buf = static_cast<const int32_t*>(bufv);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t wbase = warp * kWarpSpan + lane * 4;
    const unsigned lt = (1u << lane) - 1u;
    auto load4 = [&](int32_t pos) {
        int4 v = make_int4(-1, -1, -1, -1);
        if (BYTES) { if (pos < len) v = unpack_bytes(bufv, pos); }
        else if (VEC && pos + 3 < len) v = *reinterpret_cast<const int4*>(buf + pos);
        else {
            if (pos < len) v.x = buf[pos];
            if (pos + 1 < len) v.y = buf[pos + 1];
            if (pos + 2 < len) v.z = buf[pos + 2];
            if (pos + 3 < len) v.w = buf[pos + 3];
        }
        return v;
    };
    int cnt = 0;
#pragma unroll 4
    for (int it = 0; it < kIters; ++it) {
        const int4 v = load4(wbase + it * 128);
        cnt += (v.x == eb) + (v.y == eb) + (v.z == eb) + (v.w == eb);
    }
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0) s_cntw[warp] = cnt;
    if (tid == 0) *s_pos = 0x7fffffff;
    __syncthreads();
    int running = 0;
    for (int w = 0; w < warp; ++w) running += s_cntw[w];
    if (running <= rel && rel < running + s_cntw[warp]) {
#pragma unroll 1
        for (int it = 0; it < kIters; ++it) {
            const int32_t pos = wbase + it * 128;
            const int4 v = load4(pos);
            const bool m0 = v.x == eb, m1 = v.y == eb, m2 = v.z == eb, m3 = v.w == eb;
            const unsigned b0 = __ballot_sync(0xffffffffu, m0), b1 = __ballot_sync(0xffffffffu, m1);
            const unsigned b2 = __ballot_sync(0xffffffffu, m2), b3 = __ballot_sync(0xffffffffu, m3);
            const int tot = __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
            if (running + tot > rel) {
                int ord = running + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
                if (m0) { if (ord == rel) *s_pos = pos; ++ord; }
                if (m1) { if (ord == rel) *s_pos = pos + 1; ++ord; }
                if (m2) { if (ord == rel) *s_pos = pos + 2; ++ord; }
                if (m3) { if (ord == rel) *s_pos = pos + 3; ++ord; }
                break;
            }
            running += tot;
        }
    }
    __syncthreads();
    return *s_pos;
}

// Rewrite one chunk: `buf` holds its entries (shared memory if staged, else global memory), `tab` its table and
// `recs` its `ns` split records {expert, in-chunk ordinal of the split, target before, -} in shared memory.  Block-wide.
template <bool VEC, bool BYTES>
__device__ void rewrite_chunk(const AssignArgs& a, const void* bufv, int32_t* tab, int32_t* dst,
                              int32_t len, const int ns, int4* recs, int* s_cntw, int* s_pos)
{
    const int32_t* buf = static_cast<const int32_t*>(bufv);
    const int E = a.E;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t wbase = warp * kWarpSpan + lane * 4;
    auto emit = [&](int32_t pos, const int4& v) {
        if (VEC) st_stream(reinterpret_cast<int4*>(dst + pos), v);
        else {
            if (pos < len) dst[pos] = v.x;
            if (pos + 1 < len) dst[pos + 1] = v.y;
            if (pos + 2 < len) dst[pos + 2] = v.z;
            if (pos + 3 < len) dst[pos + 3] = v.w;
        }
    };
    auto fetch = [&](int32_t pos) {
        int4 v = make_int4(-1, -1, -1, -1);
        if (BYTES) v = unpack_bytes(bufv, pos);
        else if (VEC) v = *reinterpret_cast<const int4*>(buf + pos);
        else {
            if (pos < len) v.x = buf[pos];
            if (pos + 1 < len) v.y = buf[pos + 1];
            if (pos + 2 < len) v.z = buf[pos + 2];
            if (pos + 3 < len) v.w = buf[pos + 3];
        }
        return v;
    };
    if (ns == 0) {
        // ---- the common case: one table lookup per entry (values >= E or < 0 pass through unchanged)
#pragma unroll 4
        for (int it = 0; it < kIters; ++it) {
            const int32_t pos = wbase + it * 128;
            if (pos < len) {
                int4 v = fetch(pos);
                if (BYTES || (uint32_t)v.x < (uint32_t)E) v.x = tab[v.x];  // a staged byte is an expert
                if (BYTES || (uint32_t)v.y < (uint32_t)E) v.y = tab[v.y];
                if (BYTES || (uint32_t)v.z < (uint32_t)E) v.z = tab[v.z];
                if (BYTES || (uint32_t)v.w < (uint32_t)E) v.w = tab[v.w];
                emit(pos, v);
            }
        }
        return;
    }
    if (ns <= kFewSplits) {
        // ---- a few splits: locate each, then apply them latest position first as predicated overrides
        int32_t re[kFewSplits], rp[kFewSplits], rt[kFewSplits];
#pragma unroll
        for (int k = 0; k < kFewSplits; ++k) {
            re[k] = -1; rp[k] = -1; rt[k] = 0;            // -1 never equals a valid expert
            if (k < ns) {                                  // uniform over the block
                const int4 rec = recs[k];
                re[k] = rec.x;
                rt[k] = rec.z;
                rp[k] = locate_split<VEC, BYTES>(bufv, len, rec.x, rec.y, s_cntw, s_pos);
            }
        }
#pragma unroll
        for (int x = 1; x < kFewSplits; ++x)               // sort by position, descending (unused records sink)
#pragma unroll
            for (int y = x; y > 0; --y)
                if (rp[y] > rp[y - 1]) {
                    int32_t t;
                    t = rp[y]; rp[y] = rp[y - 1]; rp[y - 1] = t;
                    t = re[y]; re[y] = re[y - 1]; re[y - 1] = t;
                    t = rt[y]; rt[y] = rt[y - 1]; rt[y - 1] = t;
                }
        // the loop over the entries, with as many overrides per entry as the chunk has splits (the same for the block)
        auto sweep = [&](auto nsc) {
            constexpr int NS = decltype(nsc)::value;
#pragma unroll 2
            for (int it = 0; it < kIters; ++it) {
                const int32_t pos = wbase + it * 128;
                if (pos < len) {
                    int4 v = fetch(pos);
                    int32_t* xv = reinterpret_cast<int32_t*>(&v);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int32_t e = xv[j];
                        if (BYTES || (uint32_t)e < (uint32_t)E) {          // a staged byte is an expert
                            int32_t t = tab[e];
#pragma unroll
                            for (int k = 0; k < NS; ++k)
                                if (e == re[k] && pos + j < rp[k]) t = rt[k];
                            xv[j] = t;
                        }
                    }
                    emit(pos, v);
                }
            }
        };
        if (ns == 1) sweep(std::integral_constant<int, 1>{});
        else if (ns == 2) sweep(std::integral_constant<int, 2>{});
        else if (ns == 3) sweep(std::integral_constant<int, 3>{});
        else sweep(std::integral_constant<int, kFewSplits>{});
        return;
    }
    // ---- many splits in one chunk (rare): located one by one, then a list walk
    const int nrec = ns;
    for (int k = 0; k < nrec; ++k) {
        const int32_t P = locate_split<VEC, BYTES>(bufv, len, recs[k].x, recs[k].y, s_cntw, s_pos);
        if (tid == 0) recs[k].w = P;
    }
    __syncthreads();
    for (int k = tid; k < nrec; k += blockDim.x) {      // mark the experts that have a split: -1 - target
        const int32_t e = recs[k].x;
        const int32_t t = tab[e];
        if (t >= 0) tab[e] = -1 - t;
    }
    __syncthreads();
#pragma unroll 1
    for (int it = 0; it < kIters; ++it) {
        const int32_t pos = wbase + it * 128;
        if (pos < len) {
            int4 v = fetch(pos);
            int32_t* xv = reinterpret_cast<int32_t*>(&v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int32_t e = xv[j];
                if ((uint32_t)e >= (uint32_t)E) continue;
                int32_t t = tab[e];
                if (t < 0) {                               // nearest split after this position, else the final target
                    int32_t best = 0x7fffffff;
                    t = -1 - t;
                    for (int k = 0; k < nrec; ++k) {
                        const int4 r = recs[k];
                        if (r.x == e && pos + j < r.w && r.w < best) { best = r.w; t = r.z; }
                    }
                }
                xv[j] = t;
            }
            emit(pos, v);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// staging with bulk asynchronous copies

constexpr uint32_t kWaitSpins = 1u << 20;               // bound on mbarrier polling (each poll can itself block for a while)
constexpr uint32_t kBulkPiece = 8192;                   // bytes per bulk copy: several pieces in flight per chunk

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// bulk copy global -> shared with an L2 policy for data that is read once: first in line for eviction
__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_load_once(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol) : "memory");
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

// shared memory of one CTA after the staged chunk: table, this chunk's counts and starting ordinals per expert, the
// entries of the source rank (slot, expert, ordinal interval), the split records
__host__ __device__ inline size_t chunk_smem_words(int E, int S)
{
    const size_t Ep = ((size_t)E + 3) & ~(size_t)3, Sp = ((size_t)S + 3) & ~(size_t)3;
    return 3 * Ep + 4 * Sp + 4 * Sp;
}

// One CTA per chunk.  STAGE: the chunk is first copied to shared memory with bulk asynchronous copies; otherwise it
// is read from global memory (any alignment).  While the copies are in flight the CTA builds what the rewrite needs:
// the slots its source rank feeds with their ordinal intervals (X, slot experts), the ordinal each expert has reached
// at the start of the chunk (sum of the counts of the segment's earlier chunks), the table expert -> target of the
// chunk's last entry of that expert, and one split record per quota interval that ends inside the chunk.
// BYTES (with STAGE): what is staged is the chunk as one byte per entry, left by the histogram pass -- a quarter of the
// bytes; a chunk whose flag says it holds a value that is no expert is read from the table itself, without staging.
template <bool VEC, bool STAGE, bool BYTES>
__global__ void __launch_bounds__(kThreads)
assign_chunk_kernel(AssignArgs a)
{
    extern __shared__ __align__(128) unsigned char shc[];
    const int E = a.E, S = a.R * a.K;
    const int Ep = (E + 3) & ~3, Sp = (S + 3) & ~3;
    int32_t* stage = reinterpret_cast<int32_t*>(shc);                      // [TAOT_CHUNK] if STAGE
    int32_t* tab = reinterpret_cast<int32_t*>(shc + (STAGE ? (size_t)TAOT_CHUNK * (BYTES ? 1 : 4) : 0));   // [E] targets
    int32_t* cnt = tab + Ep;                             // [E] entries of each expert in this chunk
    int32_t* base = cnt + Ep;                            // [E] ordinal of each expert at the start of this chunk
    int32_t* ent_s = base + Ep;                          // [S] slots this rank feeds, ascending ...
    int32_t* ent_e = ent_s + Sp;                         //     ... their experts ...
    int32_t* ent_lo = ent_e + Sp;                        //     ... and the ordinals [lo, hi) they take
    int32_t* ent_hi = ent_lo + Sp;
    int4* recs = reinterpret_cast<int4*>(ent_hi + Sp);   // [S] split records of this chunk
    __shared__ __align__(8) uint64_t bar;
    __shared__ int s_cntw[kWarps];
    __shared__ int s_wcnt[32];
    __shared__ int s_pos;
    __shared__ int s_ns;
    const int tid = threadIdx.x;
    const int64_t id = blockIdx.x;
    const int64_t lr = id / a.nc;
    const int c = (int)(id % a.nc);
    int64_t goff; int32_t len;
    chunk_geometry(a, id, goff, len);
    const void* buf = a.topk + goff;
    if (STAGE) {
        if (tid == 0) {
            mbar_init(&bar, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            const uint32_t bytes = (uint32_t)len * (BYTES ? 1u : 4u);
            const unsigned char* from = BYTES ? a.tb + goff : reinterpret_cast<const unsigned char*>(a.topk + goff);
            mbar_expect_tx(&bar, bytes);
            const uint64_t once = policy_evict_first();
            for (uint32_t o = 0; o < bytes; o += kBulkPiece)
                bulk_load_once(reinterpret_cast<unsigned char*>(stage) + o, from + o,
                               (bytes - o) < kBulkPiece ? (bytes - o) : kBulkPiece, &bar, once);
        }
        buf = stage;
    }
    const int32_t flagged = BYTES ? a.tbflag[id] : 0;    // the staged bytes are of no use: read the table itself
    // ---- the chunk's table and split records
    if (tid == 0) s_ns = 0;
    const int32_t* ccseg = a.cc + lr * a.nc * (int64_t)E;
    for (int e = tid; e < E; e += kThreads) {
        int32_t b = 0;
        for (int cb = 0; cb < c; ++cb) b += ccseg[(int64_t)cb * E + e];
        base[e] = b;
        cnt[e] = ccseg[(int64_t)c * E + e];
        tab[e] = e;
    }
    const int m = build_entries(a.X + lr * S, a.slot_expert + (lr / a.R) * S, S, E, ent_s, ent_e, ent_lo, ent_hi, s_wcnt);
    for (int q = tid; q < m; q += kThreads) {
        const int e = ent_e[q];
        const int32_t n = cnt[e];
        if (n == 0) continue;
        const int32_t b = base[e], lo = ent_lo[q], hi = ent_hi[q];
        const int32_t last = b + n - 1;
        if (lo <= last && last < hi) tab[e] = E + ent_s[q];               // the slot that takes the chunk's last entry of e
        if (hi > b && hi < b + n)                                         // this slot's quota ends inside the chunk
            recs[atomicAdd(&s_ns, 1)] = make_int4(e, hi - b, E + ent_s[q], -1);
    }
    __syncthreads();                                     // table and records in place; the barrier is initialised
    if (STAGE) {
        const bool ok = mbar_wait(&bar, 0);
        if (__syncthreads_or(!ok)) {                     // the copy has not landed: report, and give the copies still in
            if (tid == 0) {                              // flight one more bounded wait before the CTA's memory goes away
                atomicOr(a.info + (int32_t)(lr / a.R), TAOT_INFO_INTERNAL);
                (void)mbar_wait(&bar, 0);
            }
            return;
        }
    }
    if (BYTES && flagged) rewrite_chunk<VEC, false>(a, a.topk + goff, tab, a.out + goff, len, s_ns, recs, s_cntw, &s_pos);
    else rewrite_chunk<VEC, BYTES>(a, buf, tab, a.out + goff, len, s_ns, recs, s_cntw, &s_pos);
}

}  // namespace

int taot_launch_assign(taot_handle_t h, const int32_t* d_topk, void* ws, const int32_t* d_slot_expert,
                       const int32_t* d_X, int32_t* d_new_idx, int32_t* d_info, cudaStream_t st)
{
    const taot_params& p = h->p;
    char* w = static_cast<char*>(ws);
    AssignArgs a;
    a.topk = d_topk;
    a.cc = reinterpret_cast<const int32_t*>(w + h->off_cc);
    a.slot_expert = d_slot_expert; a.X = d_X; a.out = d_new_idx; a.info = d_info;
    a.layer_elems = p.T * p.k; a.seg = h->seg; a.nc = h->nc; a.R = p.R; a.E = p.E; a.K = p.K;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(d_topk) & 15) == 0) &&
                       ((reinterpret_cast<uintptr_t>(d_new_idx) & 15) == 0) && (h->seg % 4 == 0);
    const int S = p.R * p.K;
    const unsigned blocks = (unsigned)((int64_t)p.L * p.R * h->nc);
    const size_t words = chunk_smem_words(p.E, S);
    a.tb = nullptr; a.tbflag = nullptr;
    if (vec_ok && h->tb_ok) {
        // the histogram pass that left the chunk counts also left the table as one byte per entry
        a.tb = reinterpret_cast<const uint8_t*>(w + h->off_tb);
        a.tbflag = reinterpret_cast<const int32_t*>(w + h->off_tbflag);
        const size_t smem = (size_t)TAOT_CHUNK + sizeof(int32_t) * words;
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_chunk_kernel<true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        assign_chunk_kernel<true, true, true><<<blocks, kThreads, smem, st>>>(a);
    } else if (vec_ok) {
        const size_t smem = (size_t)TAOT_CHUNK * 4 + sizeof(int32_t) * words;
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_chunk_kernel<true, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        assign_chunk_kernel<true, true, false><<<blocks, kThreads, smem, st>>>(a);
    } else {
        const size_t smem = sizeof(int32_t) * words;
        TAOT_CUDA_OK(cudaFuncSetAttribute(assign_chunk_kernel<false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        assign_chunk_kernel<false, false, false><<<blocks, kThreads, smem, st>>>(a);
    }
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
