// Sinkhorn-Knopp (Appendix A.2) for a whole batch at once on the tensor cores: the Gibbs kernel
// M = exp(-C/eps) is the same for every problem of a call, so one half-step of all B problems,
//     u = s~ / (M v)        or        v = d / (M^T u),
// is one dense product [R,R] x [R,B] followed by an element-wise divide.  This file is that product as a
// tcgen05 (UMMA) GEMM with the divide fused into its epilogue, for the case the other kernels serve worst: a
// cost matrix with no tier structure at more than 256 ranks, a fixed iteration count, and C/eps small enough
// for exp(-C/eps) and the scaling vectors to stay inside fp32 (the multiplicative form of the paper, as printed).
//
// Precision.  The tensor cores multiply TF32 (11 significant bits).  Every operand x is therefore kept as two
// TF32-exact floats, hi = x with its low 13 mantissa bits cleared and lo = (x - hi) with its low 13 bits cleared,
// and a product is accumulated (fp32, in tensor memory) as  hi*hi + hi*lo + lo*hi : three MMAs per k-step, error
// about 2^-21 per term, all terms positive.  Because hi and lo are exact TF32 values it does not matter whether
// the hardware truncates or rounds its inputs.
//
// One CTA computes one 128 x N tile of the product (128 ranks x N problems): warp 0 streams the operand tiles
// (A: rows of M or M^T, hi and lo; B: rows of v or u, hi and lo) into a ring of shared-memory stages with TMA
// (cp.async.bulk.tensor, 128-byte swizzle, each CTA loads its own tiles: no multicast), one lane of warp 1
// issues the MMAs and commits each stage back to the loader and the finished tile to the epilogue, warps 2-5 read
// the accumulator from tensor memory (each warp the 32 lanes of its quadrant), divide, split the quotient into
// hi / lo and store it in the [B,R] layout the next half-step loads as its B operand.  Every wait is bounded; a
// wait that runs out raises a flag in global memory, the CTA waits (bounded) for its copies in flight, frees its
// tensor memory and leaves.
#include <cuda.h>

#include <cstdlib>

#include "sinkhorn_common.cuh"

using namespace taot_sk;

namespace {

constexpr int kTileM = 128;                 // ranks per tile = TMEM lanes
constexpr int kBlockK = 32;                 // floats per k-block = one 128-byte swizzle row
constexpr int kUmmaK = 8;                   // TF32 MMA depth
constexpr int kTcThreads = 192;             // warp 0 loads, warp 1 issues MMAs, warps 2-5 are the epilogue
constexpr uint32_t kTcSpins = 1u << 20;     // bound on every mbarrier wait

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// false if the bound ran out
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity)
{
    const uint32_t addr = smem_addr(bar);
    for (uint32_t spin = 0; spin < kTcSpins; ++spin) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done)
                     : "r"(addr), "r"(parity)
                     : "memory");
        if (done) return true;
    }
    return false;
}

// one 2-D tile (box of the tensor map) from this GPU's global memory into shared memory; completion on `bar`
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_addr(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_addr(bar))
                 : "memory");
}

// shared-memory matrix descriptor of a K-major tile with 128-byte swizzle: rows of 128 bytes, atoms of 8 rows
// (1024 bytes apart), descriptor version 1
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// instruction descriptor: TF32 x TF32 -> F32, both operands K-major, M = 128, N columns
__host__ __device__ constexpr uint32_t umma_idesc_tf32(int n)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"      // no output lane disabled
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// arrive on `bar` once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

struct TcArgs {
    const float* num;        // [B,R] numerator of the divide: s~ for the u-update, d for the v-update
    float* out_hi;           // [B,R] quotient, TF32-exact high part
    float* out_lo;           // [B,R] TF32-exact low part
    int32_t* abort_flag;     // set if a bounded wait ran out
    int32_t R, B;
};

// The tensor cores add into their fp32 accumulator with truncation, so a long sum of positive terms comes out low by
// an amount that grows with its length (measured: plan error up to 1e-4 at 1024 ranks with one accumulator).  The
// terms are therefore dealt round-robin to kAcc accumulators (k-step j to accumulator j mod kAcc; all 512 columns of
// tensor memory are used) and the epilogue adds the accumulators in fp32 with rounding.
template <int N>
struct TcAcc {
    static constexpr int kAcc = 512 / N < 4 ? 512 / N : 4;
    static constexpr int kCols = 512;
};

template <int N>
struct TcSmem {
    static constexpr int kStageBytes = 2 * kTileM * kBlockK * 4 + 2 * N * kBlockK * 4;     // A hi, A lo, B hi, B lo
    static constexpr int kStages = (200 * 1024) / kStageBytes < 4 ? (200 * 1024) / kStageBytes : 4;
    static constexpr int kBytes = kStages * kStageBytes + 1024;                            // + room to align to 1024
};

template <int N>
__global__ void __launch_bounds__(kTcThreads, 1)
sinkhorn_tc_halfstep_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
                            const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
                            TcArgs a)
{
    using SM = TcSmem<N>;
    constexpr int kStages = SM::kStages;
    extern __shared__ unsigned char tc_smem_raw[];
    __shared__ __align__(8) uint64_t full[4], empty[4], acc_full;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;
    unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kTileM;                   // first rank of the tile
    const int n0 = blockIdx.y * N;                        // first problem of the tile
    const int nk = a.R / kBlockK;

    // a solve is a long chain of these launches: once one of them has given up, the rest return at once (the flag is
    // read by one thread and handed to the others through shared memory, so that all of them take the same way)
    if (tid == 0) s_abort = *(volatile int32_t*)a.abort_flag;
    __syncthreads();
    if (s_abort) return;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { bar_init(&full[s], 1); bar_init(&empty[s], 1); }
        bar_init(&acc_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                                      // tensor memory for the accumulator: N columns of 128 lanes
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&s_tmem)), "r"((uint32_t)TcAcc<N>::kCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = s_tmem;

    if (warp == 0) {
        // ---------------------------------------------------------------- loader
        if (lane == 0) {
            int armed = 0;                                // stages whose copies may still be in flight (bit set)
            for (int kb = 0; kb < nk; ++kb) {
                const int s = kb % kStages;
                if (kb >= kStages && !bar_wait(&empty[s], ((kb / kStages) - 1) & 1)) {
                    atomicExch(a.abort_flag, 1);
                    *(volatile int*)&s_abort = 1;
                    break;
                }
                if (*(volatile int*)&s_abort) break;
                unsigned char* st = tiles + (size_t)s * SM::kStageBytes;
                bar_expect_tx(&full[s], (uint32_t)SM::kStageBytes);
                tma_load_2d(st, &map_a_hi, kb * kBlockK, m0, &full[s]);
                tma_load_2d(st + kTileM * kBlockK * 4, &map_a_lo, kb * kBlockK, m0, &full[s]);
                tma_load_2d(st + 2 * kTileM * kBlockK * 4, &map_b_hi, kb * kBlockK, n0, &full[s]);
                tma_load_2d(st + 2 * kTileM * kBlockK * 4 + N * kBlockK * 4, &map_b_lo, kb * kBlockK, n0, &full[s]);
                armed |= 1 << s;
            }
            if (*(volatile int*)&s_abort) {
                // the MMA thread may never consume what is still landing: one more bounded wait per armed stage, on
                // either phase, before this CTA's shared memory goes away
                for (int s = 0; s < kStages; ++s)
                    if (armed & (1 << s)) { (void)bar_wait(&full[s], 0); (void)bar_wait(&full[s], 1); }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issue
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_tf32(N);
            bool ok = true;
            for (int kb = 0; kb < nk && ok; ++kb) {
                const int s = kb % kStages;
                ok = bar_wait(&full[s], (kb / kStages) & 1) && !*(volatile int*)&s_abort;
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t st = smem_addr(tiles + (size_t)s * SM::kStageBytes);
                const uint32_t a_hi = st, a_lo = st + kTileM * kBlockK * 4;
                const uint32_t b_hi = st + 2 * kTileM * kBlockK * 4, b_lo = b_hi + N * kBlockK * 4;
                // The four k-steps of a block go to different accumulators (k-step j of the whole sum to accumulator
                // j mod kAcc), and the three products of a term are issued k-step by k-step: consecutive MMAs then never
                // add into the same accumulator, which they would otherwise do one full MMA latency apart.
                constexpr int kAcc = TcAcc<N>::kAcc;
                const uint32_t fresh = kb == 0 ? 0u : 1u;
#pragma unroll
                for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                    const uint32_t off = (uint32_t)k * kUmmaK * 4;        // 32 bytes along the swizzled row
                    umma_tf32(tmem_d + (uint32_t)((k % kAcc) * N), umma_desc_sw128(a_hi + off), umma_desc_sw128(b_hi + off), idesc,
                              k < kAcc ? fresh : 1u);
                }
#pragma unroll
                for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                    const uint32_t off = (uint32_t)k * kUmmaK * 4;
                    umma_tf32(tmem_d + (uint32_t)((k % kAcc) * N), umma_desc_sw128(a_hi + off), umma_desc_sw128(b_lo + off), idesc, 1u);
                }
#pragma unroll
                for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                    const uint32_t off = (uint32_t)k * kUmmaK * 4;
                    umma_tf32(tmem_d + (uint32_t)((k % kAcc) * N), umma_desc_sw128(a_lo + off), umma_desc_sw128(b_hi + off), idesc, 1u);
                }
                umma_commit(&empty[s]);                   // the stage is free once these MMAs have read it
            }
            if (!ok) {
                atomicExch(a.abort_flag, 1);
                *(volatile int*)&s_abort = 1;
            }
            umma_commit(&acc_full);                       // (also on the way out: the epilogue's wait then ends early)
        }
    } else {
        // ---------------------------------------------------------------- epilogue: warps 2..5, TMEM quadrant warp % 4
        const int quad = warp & 3;
        const int i = m0 + quad * 32 + lane;              // this thread's rank = TMEM lane
        const bool ok = __all_sync(0xffffffffu, bar_wait(&acc_full, 0) && !*(volatile int*)&s_abort);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (!ok) {
            if (lane == 0) { atomicExch(a.abort_flag, 1); *(volatile int*)&s_abort = 1; }
        } else {
#pragma unroll 1
            for (int c0 = 0; c0 < N; c0 += 32) {
                // the chunk's global loads go out first (independent of each other; behind a store or a tensor-memory load the
                // compiler could not move them up), the accumulators are read while they are in flight
                float nu[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int b = n0 + c0 + j;
                    const size_t q = (size_t)(b < a.B ? b : 0) * a.R + i;
                    nu[j] = b < a.B ? __ldg(a.num + q) : 0.0f;
                }
                uint32_t acc[32];
                float sum[32];
                constexpr int kAcc = TcAcc<N>::kAcc;
                // parts added pairwise, with rounding: (p0 + p1) + (p2 + p3)
#pragma unroll
                for (int pp = 0; pp < kAcc; pp += 2) {
                    float pair[32];
                    tmem_load32(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(pp * N + c0), acc);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 32; ++j) pair[j] = __uint_as_float(acc[j]);
                    if (pp + 1 < kAcc) {
                        tmem_load32(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)((pp + 1) * N + c0), acc);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int j = 0; j < 32; ++j) pair[j] += __uint_as_float(acc[j]);
                    }
#pragma unroll
                    for (int j = 0; j < 32; ++j) sum[j] = pp == 0 ? pair[j] : sum[j] + pair[j];
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int b = n0 + c0 + j;
                    if (b < a.B) {
                        const size_t q = (size_t)b * a.R + i;
                        const float val = (nu[j] > 0.0f && sum[j] > 0.0f) ? __fdiv_rn(nu[j], sum[j]) : 0.0f;
                        const float hi = __uint_as_float(__float_as_uint(val) & 0xFFFFE000u);
                        const float lo = __uint_as_float(__float_as_uint(val - hi) & 0xFFFFE000u);
                        a.out_hi[q] = hi;
                        a.out_lo[q] = lo;
                    }
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"((uint32_t)TcAcc<N>::kCols) : "memory");
    }
}

}  // namespace

namespace {

// gamma-scaled supply, the starting v = 1 on every rank (Appendix A.2 uses v before it defines it: v0 = 1), flags
__global__ void __launch_bounds__(256)
tc_prepare_kernel(const float* __restrict__ s, const float* __restrict__ d, int32_t R, float eps0, float* st,
                  float* v_hi, float* v_lo, int32_t* info)
{
    __shared__ double red[2][8];
    const int64_t b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double ps = 0.0, pd = 0.0;
    for (int r = tid; r < R; r += 256) {
        const float sv = s[b * R + r], dv = d[b * R + r];
        ps += sv > 0.0f ? (double)sv : 0.0;
        pd += dv > 0.0f ? (double)dv : 0.0;
    }
    for (int o = 16; o > 0; o >>= 1) { ps += __shfl_xor_sync(0xffffffffu, ps, o); pd += __shfl_xor_sync(0xffffffffu, pd, o); }
    if (lane == 0) { red[0][warp] = ps; red[1][warp] = pd; }
    __syncthreads();
    ps = 0.0; pd = 0.0;
    for (int w = 0; w < 8; ++w) { ps += red[0][w]; pd += red[1][w]; }
    const double gamma = fmin(1.0, pd / fmax(ps, (double)eps0));
    for (int r = tid; r < R; r += 256) {
        const float sv = s[b * R + r];
        st[b * R + r] = sv > 0.0f ? (float)(gamma * (double)sv) : 0.0f;
        v_hi[b * R + r] = 1.0f;
        v_lo[b * R + r] = 0.0f;
    }
    if (tid == 0 && ps > pd) atomicOr(info + b, TAOT_INFO_SUPPLY_SCALED);
}

// T = diag(u) M diag(v) with the column cap (Appendix A.2).  One CTA writes kFinRows rows of one problem's plan and the
// sum over those rows of |row sum - s~_i| (row sums in fp64, lanes and warps added in a fixed order).
constexpr int kFinRows = 8;

__global__ void __launch_bounds__(256)
tc_finalize_kernel(const float* __restrict__ m_hi, const float* __restrict__ m_lo, const float* __restrict__ u_hi,
                   const float* __restrict__ u_lo, const float* __restrict__ v_hi, const float* __restrict__ v_lo,
                   const float* __restrict__ st, const float* __restrict__ d, int32_t R, float eps0,
                   float* __restrict__ plan, double* __restrict__ err_part, int32_t* info)
{
    __shared__ double red[8];
    const int64_t b = blockIdx.y;
    const int i0 = blockIdx.x * kFinRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int nonfinite = 0;
    double err = 0.0;
    for (int ii = 0; ii < kFinRows; ++ii) {
        const int i = i0 + ii;
        if (i >= R) break;                                  // uniform over the CTA
        const float u = u_hi[b * R + i] + u_lo[b * R + i];
        float* orow = plan + (b * R + i) * (int64_t)R;
        double rs = 0.0;
        for (int j = tid; j < R; j += 256) {
            const float dj = d[b * R + j];
            float val = 0.0f;
            if (u > 0.0f && dj > 0.0f) {
                const float v = v_hi[b * R + j] + v_lo[b * R + j];
                // after the v-update the column sums equal d, so the cap is min(1, d / (d + eps0))
                const float cap = fminf(1.0f, dj / (dj + eps0));
                val = (u * (m_hi[(int64_t)i * R + j] + m_lo[(int64_t)i * R + j])) * v * cap;
                if (!isfinite(val)) nonfinite = 1;
            }
            orow[j] = val;
            rs += (double)val;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
        if (lane == 0) red[warp] = rs;
        __syncthreads();
        if (tid == 0) {
            double tot = 0.0;
            for (int w = 0; w < 8; ++w) tot += red[w];
            err += fabs(tot - (double)st[b * R + i]);
        }
        __syncthreads();
    }
    nonfinite = __syncthreads_or(nonfinite);
    if (tid == 0) {
        err_part[b * gridDim.x + blockIdx.x] = err;
        if (nonfinite) atomicOr(info + b, TAOT_INFO_NONFINITE);
    }
}

// iteration count and row error of the returned iterate, per problem
__global__ void __launch_bounds__(128)
tc_report_kernel(const float* __restrict__ st, const float* __restrict__ d, const double* __restrict__ err_part, int32_t R,
                 int32_t B, int32_t parts, int32_t iters_done, int32_t* iters, float* row_err, int32_t* info,
                 const int32_t* abort_flag)
{
    const int64_t b = (int64_t)blockIdx.x * 128 + threadIdx.x;
    if (b >= B) return;
    double tot = 0.0, dsum = 0.0, err = 0.0;
    for (int r = 0; r < R; ++r) {
        tot += (double)st[b * R + r];
        dsum += d[b * R + r] > 0.0f ? (double)d[b * R + r] : 0.0;
    }
    for (int p = 0; p < parts; ++p) err += err_part[b * parts + p];
    const bool empty = !(tot > 0.0) || !(dsum > 0.0);
    iters[b] = empty ? 0 : iters_done;
    row_err[b] = empty ? 0.0f : (float)(err / tot);
    if (*abort_flag) atomicOr(info + b, TAOT_INFO_INTERNAL);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// tensor map of a row-major [rows, cols] fp32 matrix in this GPU's memory, box = box_rows x 32 floats, 128-byte swizzle
bool make_map(CUtensorMap* map, const float* base, int rows, int cols, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int N>
int run_tc(taot_handle_t h, const SinkArgs& a, int32_t B, float* ws, cudaStream_t st)
{
    const int R = a.R;
    const size_t BR = (size_t)B * R;
    float* u_hi = ws;
    float* u_lo = u_hi + BR;
    float* v_hi = u_lo + BR;
    float* v_lo = v_hi + BR;
    float* stl = v_lo + BR;
    const int parts = (R + kFinRows - 1) / kFinRows;
    double* err_part = reinterpret_cast<double*>(stl + BR);                 // [B][parts] (BR floats = an even count)
    int32_t* abort_flag = reinterpret_cast<int32_t*>(err_part + (size_t)parts * B);
    const float* m_hi = h->d_gibbs;
    const float* m_lo = m_hi + (size_t)R * R;
    const float* mt_hi = m_lo + (size_t)R * R;
    const float* mt_lo = mt_hi + (size_t)R * R;
    CUtensorMap map_m_hi, map_m_lo, map_mt_hi, map_mt_lo, map_u_hi, map_u_lo, map_v_hi, map_v_lo;
    if (!make_map(&map_m_hi, m_hi, R, R, kTileM) || !make_map(&map_m_lo, m_lo, R, R, kTileM) ||
        !make_map(&map_mt_hi, mt_hi, R, R, kTileM) || !make_map(&map_mt_lo, mt_lo, R, R, kTileM) ||
        !make_map(&map_u_hi, u_hi, B, R, N) || !make_map(&map_u_lo, u_lo, B, R, N) ||
        !make_map(&map_v_hi, v_hi, B, R, N) || !make_map(&map_v_lo, v_lo, B, R, N))
        return TAOT_ERR_CUDA;
    TAOT_CUDA_OK(cudaFuncSetAttribute(sinkhorn_tc_halfstep_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      TcSmem<N>::kBytes));
    TAOT_CUDA_OK(cudaMemsetAsync(abort_flag, 0, sizeof(int32_t), st));
    tc_prepare_kernel<<<B, 256, 0, st>>>(a.s, a.d, R, a.eps0, stl, v_hi, v_lo, a.info);
    TAOT_CUDA_OK(cudaGetLastError());
    const dim3 grid(R / kTileM, (B + N - 1) / N);
    TcArgs t;
    t.abort_flag = abort_flag; t.R = R; t.B = B;
    int launches = 1;
    for (int it = 0; it < a.max_iters; ++it) {
        t.num = stl; t.out_hi = u_hi; t.out_lo = u_lo;          // u = s~ / (M v)
        sinkhorn_tc_halfstep_kernel<N><<<grid, kTcThreads, TcSmem<N>::kBytes, st>>>(map_m_hi, map_m_lo, map_v_hi, map_v_lo, t);
        t.num = a.d; t.out_hi = v_hi; t.out_lo = v_lo;          // v = d / (M^T u)
        sinkhorn_tc_halfstep_kernel<N><<<grid, kTcThreads, TcSmem<N>::kBytes, st>>>(map_mt_hi, map_mt_lo, map_u_hi, map_u_lo, t);
        launches += 2;
    }
    TAOT_CUDA_OK(cudaGetLastError());
    const dim3 fgrid(parts, B);
    tc_finalize_kernel<<<fgrid, 256, 0, st>>>(m_hi, m_lo, u_hi, u_lo, v_hi, v_lo, stl, a.d, R, a.eps0, a.plan, err_part, a.info);
    tc_report_kernel<<<(B + 127) / 128, 128, 0, st>>>(stl, a.d, err_part, R, B, parts, a.max_iters, a.iters, a.row_err, a.info,
                                                      abort_flag);
    TAOT_CUDA_OK(cudaGetLastError());
    return launches + 2;
}

}  // namespace

// floats of workspace the tensor-core solve needs for a batch of B problems of R ranks
size_t taot_sinkhorn_tc_ws_floats(int32_t R, int32_t B)
{
    return 5 * (size_t)B * R + 2 * (size_t)((R + kFinRows - 1) / kFinRows) * B + 64;
}

// The whole fixed-count solve of a batch on the tensor cores, or 0 launches if this call is not its case (the caller
// then takes the other kernels): more than 256 ranks in multiples of 128, a handle whose Gibbs kernel fits fp32
// (taot_create built it), no tolerance test, and a batch large enough to fill the GPU with tiles.
int taot_launch_sinkhorn_dense_tc(taot_handle_t h, const SinkArgs& a, int32_t B, float* ws_tc, cudaStream_t st)
{
    if (!h->d_gibbs || !ws_tc || a.tol > 0.0f || a.R <= 256 || a.R % kTileM != 0 || B < 256 || B > h->p.L) return 0;
    const int sms = h->sm_count;
    const int mt = a.R / kTileM;
    if (const char* env = std::getenv("TAOT_TC_TILE_N")) {       // tuning knob: force the tile width
        const int n = std::atoi(env);
        if (n == 256) return run_tc<256>(h, a, B, ws_tc, st);
        if (n == 128) return run_tc<128>(h, a, B, ws_tc, st);
        if (n == 64) return run_tc<64>(h, a, B, ws_tc, st);
    }
    // (256 problems per tile is faster still but leaves room for two accumulators only: twice the truncation error)
    if (mt * ((B + 127) / 128) >= sms) return run_tc<128>(h, a, B, ws_tc, st);
    return run_tc<64>(h, a, B, ws_tc, st);
}
