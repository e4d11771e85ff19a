// Load collection (Appendix A.1): per-chunk expert histograms of the routing table, then one
// merge per layer into n[r][e], expert_load, rank_load and the excess / spare vectors.
//
// The routing table of one layer is R contiguous segments (one per source rank) of SEG = (T/R)*k
// int32 each, so n[l][r][:] is simply the E-bin histogram of segment (l, r).  Each CTA owns one
// chunk of at most TAOT_CHUNK elements of one segment: it streams the chunk with 16-byte loads,
// counts into per-warp private shared-memory histograms, and stores its E counts with plain
// stores -- no global atomics, no zero-fill of the outputs.  The per-chunk counts are kept: the
// reassignment kernel turns them into each chunk's starting ordinals.  Where the table has at most
// 256 experts the pass also leaves every entry as one byte in the workspace (plus one flag per
// chunk for values that are no expert): the reassignment, which runs last and alone on the memory
// system, then reads a quarter of the bytes, for one more byte per entry written here.
#include <cstring>
#include <mutex>

#include "taot_internal.cuh"

namespace {

constexpr int kThreads = TAOT_STREAM_THREADS;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ int4 ld_stream(const int4* p)
{
    int4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// EXTRA == false: out-of-range values are only flagged; true: they are also counted, in bin E (rows of E + 1 bins)
template <bool EXTRA>
__device__ __forceinline__ void count_one(int32_t* hist, int32_t e, int32_t E, int& bad)
{
    if ((uint32_t)e < (uint32_t)E) atomicAdd(hist + e, 1);
    else { bad = 1; if (EXTRA) atomicAdd(hist + E, 1); }
}

// four entries as four bytes (E <= 256; a value that is no expert leaves a byte nobody reads: its chunk is flagged)
__device__ __forceinline__ uint32_t pack_bytes(const int4& x)
{
    return ((uint32_t)x.x & 255u) | (((uint32_t)x.y & 255u) << 8) | (((uint32_t)x.z & 255u) << 16) | ((uint32_t)x.w << 24);
}

// tb (may be null; only with vec_ok): the table again as one byte per entry, written beside the counts, and tbflag:
// one word per chunk, nonzero if the chunk holds a value that is no expert.  The reassignment reads these 1-byte
// entries instead of the table (a quarter of the bytes) wherever the chunk's flag is zero.
template <bool EXTRA>
__global__ void __launch_bounds__(kThreads)
hist_chunk_kernel(const int32_t* __restrict__ topk, int32_t* __restrict__ cc, int32_t* __restrict__ info,
                  int64_t layer_elems, int64_t seg, int32_t nc, int32_t R, int32_t E, int vec_ok,
                  uint8_t* __restrict__ tb, int32_t* __restrict__ tbflag)
{
    const int32_t nb = EXTRA ? E + 1 : E;
    extern __shared__ int32_t sh_hist[];                 // [kWarps][nb]
    const int tid = threadIdx.x, warp = tid >> 5;
    const int64_t id = blockIdx.x;
    const int32_t c = (int32_t)(id % nc);
    const int64_t lr = id / nc;
    const int32_t l = (int32_t)(lr / R);
    const int32_t r = (int32_t)(lr % R);
    const int64_t start = (int64_t)c * TAOT_CHUNK;
    const int32_t len = (int32_t)((seg - start) < (int64_t)TAOT_CHUNK ? (seg - start) : (int64_t)TAOT_CHUNK);
    const int32_t* src = topk + (int64_t)l * layer_elems + (int64_t)r * seg + start;
    uint32_t* tb4 = (!EXTRA && tb) ? reinterpret_cast<uint32_t*>(tb + (int64_t)l * layer_elems + (int64_t)r * seg + start) : nullptr;

    for (int i = tid; i < kWarps * nb; i += kThreads) sh_hist[i] = 0;
    __syncthreads();
    int32_t* hist = sh_hist + warp * nb;
    int bad = 0;

    if (vec_ok) {
        const int4* src4 = reinterpret_cast<const int4*>(src);
        const int32_t nvec = len >> 2;
        int32_t v = tid;
        // full rounds of 8 loads in flight per thread
        for (; v + 7 * kThreads < nvec; v += 8 * kThreads) {
            int4 x[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) x[u] = ld_stream(src4 + v + u * kThreads);
            if (!EXTRA && tb4) {
#pragma unroll
                for (int u = 0; u < 8; ++u) tb4[v + u * kThreads] = pack_bytes(x[u]);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                count_one<EXTRA>(hist, x[u].x, E, bad); count_one<EXTRA>(hist, x[u].y, E, bad);
                count_one<EXTRA>(hist, x[u].z, E, bad); count_one<EXTRA>(hist, x[u].w, E, bad);
            }
        }
        for (; v < nvec; v += kThreads) {
            const int4 x = ld_stream(src4 + v);
            if (!EXTRA && tb4) tb4[v] = pack_bytes(x);
            count_one<EXTRA>(hist, x.x, E, bad); count_one<EXTRA>(hist, x.y, E, bad);
            count_one<EXTRA>(hist, x.z, E, bad); count_one<EXTRA>(hist, x.w, E, bad);
        }
        for (int32_t i = (nvec << 2) + tid; i < len; i += kThreads) count_one<EXTRA>(hist, src[i], E, bad);
    } else {
        for (int32_t i = tid; i < len; i += kThreads) count_one<EXTRA>(hist, src[i], E, bad);
    }
    const int any_bad = __syncthreads_or(bad);
    int32_t* out = cc + id * nb;
    for (int e = tid; e < nb; e += kThreads) {
        int32_t tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += sh_hist[w * nb + e];
        out[e] = tot;
    }
    if (any_bad && tid == 0) atomicOr(info + l, TAOT_INFO_BAD_INDEX);
    if (!EXTRA && tbflag && tid == 0) tbflag[id] = any_bad;
}

// excess / spare of one row of rank loads held in shared memory (Appendix A.1, integer mean)
__device__ void excess_spare_row(const int32_t* s_rl, int32_t R, long long* s_tot, int32_t* excess,
                                 int32_t* spare, float* fs, float* fd)
{
    const int tid = threadIdx.x;
    if (tid == 0) *s_tot = 0;
    __syncthreads();
    long long part = 0;
    for (int r = tid; r < R; r += blockDim.x) part += s_rl[r];
    if (part) atomicAdd(reinterpret_cast<unsigned long long*>(s_tot), (unsigned long long)part);
    __syncthreads();
    const long long m = *s_tot / R;
    for (int r = tid; r < R; r += blockDim.x) {
        const long long lr = s_rl[r];
        const int32_t ex = (int32_t)(lr > m ? lr - m : 0);
        const int32_t sp = (int32_t)(m > lr ? m - lr : 0);
        if (excess) excess[r] = ex;
        if (spare) spare[r] = sp;
        if (fs) fs[r] = (float)ex;
        if (fd) fd[r] = (float)sp;
    }
}

// n = sum over chunks, expert_load = sum over ranks, rank_load by home rank.  `parts` CTAs share a layer, each taking a
// block of source ranks; a part leaves its expert loads in part_el and counts itself done, and the part that finds
// itself last adds them up and finishes the layer (no CTA waits for another).  parts == 1: one CTA per layer, no
// exchange.  The kernel sits in the chain of latency-bound stages, so what counts is how long one layer takes.
__global__ void __launch_bounds__(1024)
merge_kernel(const int32_t* __restrict__ cc, const int32_t* __restrict__ e2r, int32_t* __restrict__ n,
             int32_t* __restrict__ expert_load, int32_t* __restrict__ rank_load, int32_t* excess,
             int32_t* spare, float* fs, float* fd, int32_t R, int32_t E, int32_t nc, int32_t* info,
             int32_t parts, int32_t* part_el, int32_t* part_cnt)
{
    extern __shared__ int32_t sh[];                      // el[E], rl[R]
    __shared__ long long s_tot;
    __shared__ int s_last;
    int32_t* s_el = sh;
    int32_t* s_rl = sh + E;
    const int l = blockIdx.x / parts, part = blockIdx.x - l * parts, tid = threadIdx.x;
    for (int i = tid; i < E + R; i += blockDim.x) sh[i] = 0;
    __syncthreads();
    const int32_t RE = R * E;                            // at most 256 x 1024
    const int32_t* ccl = cc + (int64_t)l * RE * nc;
    int32_t* nl = n + (int64_t)l * RE;
    // (32-bit index arithmetic and several independent loads in flight per thread)
    const int32_t i0 = (int32_t)((int64_t)RE * part / parts), i1 = (int32_t)((int64_t)RE * (part + 1) / parts);
#pragma unroll 4
    for (int32_t idx = i0 + tid; idx < i1; idx += blockDim.x) {
        const int32_t r = idx / E, e = idx - r * E;
        const int32_t* p = ccl + r * nc * E + e;
        int32_t v = 0;
        for (int c = 0; c < nc; ++c) v += __ldg(p + c * E);
        nl[idx] = v;
        if (v) atomicAdd(s_el + e, v);
    }
    __syncthreads();
    if (parts > 1) {
        int32_t* mine = part_el + ((int64_t)l * parts + part) * E;
        for (int e = tid; e < E; e += blockDim.x) mine[e] = s_el[e];
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = atomicAdd(part_cnt + l, 1) == parts - 1;
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        const int32_t* all = part_el + (int64_t)l * parts * E;
        for (int e = tid; e < E; e += blockDim.x) {
            int32_t v = 0;
            for (int q = 0; q < parts; ++q) v += __ldcg(all + (int64_t)q * E + e);   // written by other CTAs: not through L1
            s_el[e] = v;
        }
        if (tid == 0) part_cnt[l] = 0;                   // as the next call expects it
        __syncthreads();
    }
    for (int e = tid; e < E; e += blockDim.x) {
        const int32_t v = s_el[e];
        expert_load[(int64_t)l * E + e] = v;
        // a handle's map was validated on the host; a caller-supplied device map (the entry point without a handle)
        // was not: an expert whose home rank is out of range is left out of the rank loads and flagged
        const uint32_t home = (uint32_t)e2r[e];
        if (home < (uint32_t)R) {
            if (v) atomicAdd(s_rl + home, v);
        } else if (info) {
            atomicOr(info + l, TAOT_INFO_BAD_INDEX);
        }
    }
    __syncthreads();
    for (int r = tid; r < R; r += blockDim.x) rank_load[(int64_t)l * R + r] = s_rl[r];
    excess_spare_row(s_rl, R, &s_tot, excess ? excess + (int64_t)l * R : nullptr,
                     spare ? spare + (int64_t)l * R : nullptr, fs ? fs + (int64_t)l * R : nullptr,
                     fd ? fd + (int64_t)l * R : nullptr);
}

__global__ void __launch_bounds__(256)
excess_spare_kernel(const int32_t* __restrict__ rank_load, int32_t* excess, int32_t* spare, float* fs,
                    float* fd, int32_t R)
{
    extern __shared__ int32_t sh[];                      // rl[R]
    __shared__ long long s_tot;
    const int64_t b = blockIdx.x;
    for (int r = threadIdx.x; r < R; r += blockDim.x) sh[r] = rank_load[b * R + r];
    __syncthreads();
    excess_spare_row(sh, R, &s_tot, excess ? excess + b * R : nullptr, spare ? spare + b * R : nullptr,
                     fs ? fs + b * R : nullptr, fd ? fd + b * R : nullptr);
}

}  // namespace

namespace {

// The table as one byte per entry, as a pass of its own: a grid of a few CTAs that walks the whole table, for use while
// other streams run latency-bound kernels that want SMs to themselves (its dynamic shared memory is only there to keep
// such CTAs off the SMs it sits on, and it off theirs).
constexpr int kBytesCtas = 48;
constexpr int kBytesSmem = 100 * 1024;

__global__ void __launch_bounds__(1024)
table_bytes_kernel(const int4* __restrict__ src, uint32_t* __restrict__ dst, int64_t nvec)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; v + 3 * stride < nvec; v += 4 * stride) {
        int4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = ld_stream(src + v + u * stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) dst[v + u * stride] = pack_bytes(x[u]);
    }
    for (; v < nvec; v += stride) dst[v] = pack_bytes(ld_stream(src + v));
}

}  // namespace

int taot_launch_table_bytes(taot_handle_t h, const int32_t* d_topk, void* ws, cudaStream_t st)
{
    const taot_params& p = h->p;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(d_topk) & 15) == 0) && (h->seg % 4 == 0);
    if (!ws || !h->tb_ok || !vec_ok) return 0;
    const int64_t nvec = (int64_t)p.L * p.T * p.k / 4;
    TAOT_CUDA_OK(cudaFuncSetAttribute(table_bytes_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBytesSmem));
    table_bytes_kernel<<<kBytesCtas, 1024, kBytesSmem, st>>>(reinterpret_cast<const int4*>(d_topk),
                                                              reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + h->off_tb), nvec);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

int taot_launch_histogram(taot_handle_t h, const int32_t* d_topk, int32_t* d_cc, int32_t* d_info, cudaStream_t st,
                          void* ws, bool write_bytes)
{
    const taot_params& p = h->p;
    const int64_t layer_elems = p.T * p.k;
    const int64_t blocks = (int64_t)p.L * p.R * h->nc;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(d_topk) & 15) == 0) && (h->seg % 4 == 0);
    const size_t smem = sizeof(int32_t) * kWarps * p.E;
    // with a workspace (and 16-byte accesses) the pass also leaves the table as one byte per entry for the reassignment
    const bool bytes = ws && h->tb_ok && vec_ok;
    uint8_t* tb = (bytes && write_bytes) ? reinterpret_cast<uint8_t*>(static_cast<char*>(ws) + h->off_tb) : nullptr;
    int32_t* tbflag = bytes ? reinterpret_cast<int32_t*>(static_cast<char*>(ws) + h->off_tbflag) : nullptr;
    hist_chunk_kernel<false><<<(unsigned)blocks, kThreads, smem, st>>>(d_topk, d_cc, d_info, layer_elems, h->seg,
                                                                        h->nc, p.R, p.E, vec_ok, tb, tbflag);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

// The same chunk histogram over `bins` values with one more bin for everything out of range (rows of bins + 1
// counts): the counting pass of the dispatch metadata, where the table holds experts and guest slots.
int taot_launch_chunk_counts(taot_handle_t h, const int32_t* d_idx, int32_t* d_counts, int32_t* d_info, int32_t bins,
                             cudaStream_t st)
{
    const taot_params& p = h->p;
    const int64_t blocks = (int64_t)p.L * p.R * h->nc;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(d_idx) & 15) == 0) && (h->seg % 4 == 0);
    const size_t smem = sizeof(int32_t) * kWarps * (size_t)(bins + 1);
    // the default limit is 48 KB
    if (smem > 48 * 1024)
        TAOT_CUDA_OK(cudaFuncSetAttribute(hist_chunk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    hist_chunk_kernel<true><<<(unsigned)blocks, kThreads, smem, st>>>(d_idx, d_counts, d_info, p.T * p.k, h->seg, h->nc,
                                                                       p.R, bins, vec_ok, nullptr, nullptr);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

int taot_launch_merge(taot_handle_t h, const int32_t* d_cc, int32_t* d_n, int32_t* d_expert_load,
                      int32_t* d_rank_load, int32_t* d_excess, int32_t* d_spare, float* d_s, float* d_d,
                      cudaStream_t st, int32_t* d_info)
{
    const taot_params& p = h->p;
    const size_t smem = sizeof(int32_t) * (p.E + p.R);
    const int parts = (h->d_merge_part && h->d_merge_cnt) ? TAOT_MERGE_PARTS : 1;
    merge_kernel<<<p.L * parts, 1024, smem, st>>>(d_cc, h->d_e2r, d_n, d_expert_load, d_rank_load, d_excess, d_spare,
                                                  d_s, d_d, p.R, p.E, h->nc, d_info, parts, h->d_merge_part,
                                                  h->d_merge_cnt);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

int taot_launch_excess_spare(taot_handle_t h, const int32_t* d_rank_load, int32_t B, int32_t* d_excess,
                             int32_t* d_spare, float* d_s, float* d_d, cudaStream_t st)
{
    const taot_params& p = h->p;
    excess_spare_kernel<<<B, 256, sizeof(int32_t) * p.R, st>>>(d_rank_load, d_excess, d_spare, d_s, d_d, p.R);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

// ---------------------------------------------------------------------------------------------
// Load collection for callers that cannot allocate device memory.
//
// taot_histogram needs a caller-supplied workspace for its per-chunk counts.  A caller that sits
// inside someone else's memory plan -- a plug-in of a serving runtime whose device memory is fully
// pre-carved, code running between the stages of a captured step, a process whose memory pool is
// already exhausted -- may have no way of getting one: cudaMalloc is off limits there (it can
// fail, it synchronises the device, and it is illegal during stream capture).  For those callers
// the per-chunk counts live in the fixed array below, which is part of the library image: every GPU
// that loads libtaot.so carries these 4 MiB until the process exits, whether or not the entry point
// is ever called.
namespace {

static __device__ __align__(256) unsigned char g_static_counts[TAOT_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
int32_t* g_static_counts_addr[kMaxDevices] = {nullptr};   // device address of g_static_counts, per device

}  // namespace

extern "C" int taot_histogram_static(const int32_t* d_topk, int32_t L, int64_t T, int32_t k, int32_t R,
                                     int32_t E, const int32_t* d_e2r, int32_t* d_n, int32_t* d_expert_load,
                                     int32_t* d_rank_load, int32_t* d_info, void* stream)
{
    if (!d_topk || !d_e2r || !d_n || !d_expert_load || !d_rank_load || !d_info) return TAOT_ERR_NULL;
    if (L < 1 || R < 1 || E < 1 || k < 1 || T < R || T % R != 0 || T * (int64_t)k >= ((int64_t)1 << 31))
        return TAOT_ERR_PARAM;
    if (R > 256 || E > 1024 || k > 64) return TAOT_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(d_topk) & 3) return TAOT_ERR_ALIGN;
    const int64_t seg = T / R * k;
    const int64_t nc = (seg + TAOT_CHUNK - 1) / TAOT_CHUNK;
    const int64_t need = (int64_t)L * R * nc * E * (int64_t)sizeof(int32_t);
    if (need > (int64_t)TAOT_STATIC_SCRATCH_BYTES) return TAOT_ERR_STATIC_CAPACITY;

    // Set-up, once per device, with that device current: in host code `g_static_counts` is only a
    // stand-in for the symbol, so the address a kernel can use has to be asked for.
    int dev = -1;
    TAOT_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return TAOT_ERR_UNSUPPORTED;
    int32_t* counts = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_counts_addr[dev]) {
            void* addr = nullptr;
            if (cudaGetSymbolAddress(&addr, g_static_counts) != cudaSuccess || !addr) return TAOT_ERR_CUDA;
            g_static_counts_addr[dev] = static_cast<int32_t*>(addr);
        }
        counts = g_static_counts_addr[dev];
    }

    // The kernels are the ones taot_histogram runs; they read only these fields of a handle.
    taot_handle_s view;
    std::memset(&view, 0, sizeof(view));
    view.p.L = L; view.p.R = R; view.p.E = E; view.p.k = k; view.p.T = T;
    view.seg = seg;
    view.nc = (int32_t)nc;
    view.d_e2r = const_cast<int32_t*>(d_e2r);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Nothing in the array has to start at zero: every chunk's CTA overwrites all E of its counts
    // with plain stores before the merge kernel reads them.
    int a = taot_launch_histogram(&view, d_topk, counts, d_info, st);
    if (a < 0) return a;
    int b = taot_launch_merge(&view, counts, d_n, d_expert_load, d_rank_load, nullptr, nullptr, nullptr, nullptr, st,
                              d_info);
    if (b < 0) return b;
    return TAOT_OK;
}
