// Phase 1 for problems too large for one CTA's shared memory (more than 256 ranks): a thread-block CLUSTER of four
// CTAs per problem.  The absorbed kernel matrix K~ (|hot| x |cold| fp32, 350 KB at 1024 ranks) is split by rows
// over the four CTAs' shared memory, so an iteration never touches L2 or HBM:
//   half-step 1  each CTA forms the row sums of its own rows (a warp per row) and u~ for them;
//   half-step 2  each CTA forms the partial column sums over its rows and stores them into ALL four CTAs' shared
//                memory (remote stores through distributed shared memory: nobody waits for a round trip); after one
//                cluster barrier every CTA adds the four partials of every column in rank order from its own
//                copy (so all four get the same bits) and forms the whole v~; the row-error partials and the range
//                flags of half-step 1 travel in the same blocks, double-buffered so that one barrier per
//                iteration is enough.
// Everything else (compaction, potentials, first iteration in the log domain) is computed redundantly and
// identically by the four CTAs, which keeps every decision (stop, fold, hand back) uniform over the cluster.
// A problem whose slice does not fit, or whose fp32 sums leave the safe range, is handed back (iters = -1) to the
// shared-memory kernel with the matrix in workspace, which holds anything.
#include <cooperative_groups.h>

#include "sinkhorn_common.cuh"

namespace cg = cooperative_groups;
using namespace taot_sk;

namespace {

constexpr int kCluster = 4;
constexpr int kNT = 1024;
constexpr int kNW = kNT / 32;
constexpr int kXTail = 4;            // floats after the column partials: row-error partial, flags

struct CSmem {
    double* alpha;   // [R] by compact hot index (all rows)
    double* beta;    // [R] by compact cold index
    double* phin;    // [R] scratch
    double* red;     // [64]
    float* st;       // [R] scaled supply, compact
    float* dd;       // [R] demand, compact
    float* u;        // [R] committed u~ (own rows are current; others unused)
    float* un;       // [R]
    float* v;        // [R]
    float* vn;       // [R]
    float* xbuf;     // [2][kCluster][R + kXTail] exchange blocks, one per source CTA: partial column sums, error partial, flags
    float* errw;     // [32]
    int32_t* hot;    // [R]
    int32_t* cold;   // [R]
    int32_t* wcnt;   // [32]
    int32_t* flags;  // [4]
    float* Ks;       // [kcap] this CTA's rows of K~
};

__host__ __device__ inline size_t csmem_state_bytes(int R)
{
    return sizeof(double) * (3 * (size_t)R + 64) + sizeof(float) * (6 * (size_t)R + 2 * kCluster * ((size_t)R + kXTail) + 32) +
           sizeof(int32_t) * (2 * (size_t)R + 36);
}

__device__ __forceinline__ CSmem ccarve(unsigned char* base, int R)
{
    CSmem m;
    double* dp = reinterpret_cast<double*>(base);
    m.alpha = dp; dp += R;
    m.beta = dp; dp += R;
    m.phin = dp; dp += R;
    m.red = dp; dp += 64;
    float* fp = reinterpret_cast<float*>(dp);
    m.st = fp; fp += R;
    m.dd = fp; fp += R;
    m.u = fp; fp += R;
    m.un = fp; fp += R;
    m.v = fp; fp += R;
    m.vn = fp; fp += R;
    m.xbuf = fp; fp += 2 * kCluster * (R + kXTail);
    m.errw = fp; fp += 32;
    int32_t* ip = reinterpret_cast<int32_t*>(fp);
    m.hot = ip; ip += R;
    m.cold = ip; ip += R;
    m.wcnt = ip; ip += 32;
    m.flags = ip; ip += 4;
    m.Ks = reinterpret_cast<float*>(ip);
    return m;
}

// ordered compaction of {i < R : val[i] > 0} into list[]; returns the count (block-wide)
__device__ int compact_list(const float* val, int R, int32_t* list, int32_t* wcnt)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int total = 0;
    for (int base = 0; base < R; base += kNT) {
        const int i = base + tid;
        const bool p = (i < R) && (val[i] > 0.0f);
        const unsigned mk = __ballot_sync(0xffffffffu, p);
        if (lane == 0) wcnt[warp] = __popc(mk);
        __syncthreads();
        int off = total;
        for (int w = 0; w < warp; ++w) off += wcnt[w];
        if (p) list[off + __popc(mk & ((1u << lane) - 1u))] = i;
        for (int w = 0; w < kNW; ++w) total += wcnt[w];
        __syncthreads();
    }
    return total;
}

__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kNT, 1)
sinkhorn_cluster_kernel(SinkArgs a, int32_t kcap)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int R = a.R, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    CSmem m = ccarve(smem_raw, R);
    const int64_t b = blockIdx.x / kCluster;
    __shared__ double s_sum[2];
    const int XS = R + kXTail;                               // floats per exchange buffer

    // ---- supply scaling gamma = min(1, sum d / max(sum s, eps0)), compaction (every CTA, identically)
    {
        double ps = 0.0, pd = 0.0;
        for (int i = tid; i < R; i += kNT) {
            const float sv = a.s[b * R + i], dv = a.d[b * R + i];
            ps += sv > 0.0f ? (double)sv : 0.0;
            pd += dv > 0.0f ? (double)dv : 0.0;
        }
        for (int o = 16; o > 0; o >>= 1) {
            ps += __shfl_xor_sync(0xffffffffu, ps, o);
            pd += __shfl_xor_sync(0xffffffffu, pd, o);
        }
        if (lane == 0) { m.red[warp] = ps; m.red[32 + warp] = pd; }
        __syncthreads();
        if (tid == 0) {
            double S = 0.0, D = 0.0;
            for (int w = 0; w < kNW; ++w) { S += m.red[w]; D += m.red[32 + w]; }
            s_sum[0] = S; s_sum[1] = D;
        }
        __syncthreads();
    }
    const double sum_s = s_sum[0], sum_d = s_sum[1];
    const double gamma = fmin(1.0, sum_d / fmax(sum_s, (double)a.eps0));
    for (int i = tid; i < R; i += kNT) {
        const float sv = a.s[b * R + i], dv = a.d[b * R + i];
        m.un[i] = sv > 0.0f ? (float)(gamma * (double)sv) : 0.0f;
        m.vn[i] = dv > 0.0f ? dv : 0.0f;
    }
    __syncthreads();
    const int Hn = compact_list(m.un, R, m.hot, m.wcnt);
    const int Cn = compact_list(m.vn, R, m.cold, m.wcnt);
    for (int i = tid; i < Hn; i += kNT) m.st[i] = m.un[m.hot[i]];
    for (int j = tid; j < Cn; j += kNT) m.dd[j] = m.vn[m.cold[j]];
    __syncthreads();

    // this CTA's rows of the compact problem
    const int per = (Hn + kCluster - 1) / kCluster;
    const int i0 = min(Hn, rank * per), i1 = min(Hn, i0 + per);
    int info = 0;
    if (sum_s > sum_d) info |= TAOT_INFO_SUPPLY_SCALED;
    float* out = a.plan + b * (int64_t)R * R;

    if (Hn == 0 || Cn == 0 || (int64_t)per * Cn > (int64_t)kcap) {       // uniform over the cluster
        if (Hn == 0 || Cn == 0) {
            for (int64_t q = (int64_t)rank * kNT + tid; q < (int64_t)R * R; q += (int64_t)kCluster * kNT) out[q] = 0.0f;
            if (rank == 0 && tid == 0) {
                a.iters[b] = 0;
                a.row_err[b] = 0.0f;
                if (info) atomicOr(a.info + b, info);
            }
        } else if (rank == 0 && tid == 0) {
            a.iters[b] = kHandBack;                                      // slice too large: the other kernel takes it
        }
        return;
    }
    // every CTA of the cluster must be running before any of them writes into another's shared memory; the
    // early return above is taken by all four or by none, so all four reach this barrier
    cluster.sync();

    double sum_st = 0.0;
    for (int i = 0; i < Hn; ++i) sum_st += (double)m.st[i];              // same order in every thread
    const double tol_abs = (double)a.tol * sum_st;

    auto rebuild = [&]() {                                               // own rows of K~ from the potentials
        const int n = (i1 - i0) * Cn;
        for (int q = tid; q < n; q += kNT) {
            const int il = q / Cn, j = q - il * Cn;
            const double c = (double)a.C[(int64_t)m.hot[i0 + il] * R + m.cold[j]] * a.inv_eps;
            m.Ks[q] = exp_split(m.alpha[i0 + il] + m.beta[j] - c);
        }
    };

    // ---- iteration 1 in the log domain (v = 1 on every rank): phi = log s~ - LSE_j(-C_ij/eps) over all j,
    //      psi_j = log d_j - LSE_i(phi_i - C_ij/eps); every CTA computes all of it
    for (int i = tid; i < Hn; i += kNT) {
        m.phin[i] = log((double)m.st[i]) - a.rowlse0[m.hot[i]];
        m.u[i] = 1.0f;
    }
    __syncthreads();
    for (int j = tid; j < Cn; j += kNT) {
        const int cj = m.cold[j];
        double mx = -INFINITY;
        for (int i = 0; i < Hn; ++i) {
            const double x = m.phin[i] - (double)a.C[(int64_t)m.hot[i] * R + cj] * a.inv_eps;
            mx = x > mx ? x : mx;
        }
        double acc = 0.0;
        for (int i = 0; i < Hn; ++i)
            acc += (double)exp_split(m.phin[i] - (double)a.C[(int64_t)m.hot[i] * R + cj] * a.inv_eps - mx);
        m.beta[j] = log((double)m.dd[j]) - (mx + log(acc));
        m.v[j] = 1.0f;
        m.vn[j] = 1.0f;
    }
    for (int i = tid; i < Hn; i += kNT) m.alpha[i] = m.phin[i];
    __syncthreads();
    rebuild();
    __syncthreads();

    int t = 1;
    float err_out = 0.0f;
    bool handed_back = false;
    // committed and candidate vectors swap roles on every commit, so an iteration needs no copy and only two block
    // barriers besides the cluster barrier
    float* ucur = m.u; float* unew = m.un;
    float* vcur = m.v; float* vnew = m.vn;
    if (tid < 4) m.flags[tid] = 0;
    __syncthreads();
    for (;;) {
        float* xb = m.xbuf + (t & 1) * kCluster * XS;      // this iteration's blocks: [source rank][XS], filled by the peers
        float* xd[kCluster];                                // my block inside every CTA's copy (remote stores)
#pragma unroll
        for (int k = 0; k < kCluster; ++k) xd[k] = cluster.map_shared_rank(xb, k) + rank * XS;
        // ================= half-step 1 (own rows): r = K~ v~, u' = s~ / r, row error of iterate t
        {
            float e = 0.0f;
            for (int i = i0 + warp; i < i1; i += kNW) {
                const float* krow = m.Ks + (i - i0) * Cn;
                float pa = 0.0f, pb = 0.0f;
                int j = lane;
                for (; j + 32 < Cn; j += 64) { pa = fmaf(krow[j], vcur[j], pa); pb = fmaf(krow[j + 32], vcur[j + 32], pb); }
                if (j < Cn) pa = fmaf(krow[j], vcur[j], pa);
                float p = pa + pb;
                for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
                if (lane == 0) {
                    if (!(p > kSumLo && p < kSumHi)) m.flags[0] = 1;
                    const float un = m.st[i] / p;
                    if (!(un > kDriftLo && un < kDriftHi)) m.flags[1] = 1;
                    unew[i] = un;
                    e += fabsf(fmaf(ucur[i], p, -m.st[i]));
                }
            }
            if (lane == 0) m.errw[warp] = e;
        }
        __syncthreads();
        // ================= half-step 2, partial over own rows; error partial and flags ride along
        for (int j = tid; j < Cn; j += kNT) {
            // four independent accumulators over the rows (summed in a fixed order): the loop is latency-bound otherwise
            float p0 = 0.0f, p1 = 0.0f, p2 = 0.0f, p3 = 0.0f;
            const float* kc = m.Ks + j;
            const float* ur = unew + i0;
            const int n = i1 - i0;
            int i = 0;
            for (; i + 3 < n; i += 4) {
                p0 = fmaf(kc[(i + 0) * Cn], ur[i + 0], p0);
                p1 = fmaf(kc[(i + 1) * Cn], ur[i + 1], p1);
                p2 = fmaf(kc[(i + 2) * Cn], ur[i + 2], p2);
                p3 = fmaf(kc[(i + 3) * Cn], ur[i + 3], p3);
            }
            for (; i < n; ++i) p0 = fmaf(kc[i * Cn], ur[i], p0);
            const float p = (p0 + p1) + (p2 + p3);
#pragma unroll
            for (int k = 0; k < kCluster; ++k) xd[k][j] = p;             // pushed, so that the reads after the barrier are local
        }
        if (warp == 0) {
            float e = m.errw[lane];                                      // one partial per warp, reduced in a fixed tree
            for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
            if (lane == 0) {
                const float fl0 = __int_as_float(m.flags[0] | (m.flags[1] << 1));
#pragma unroll
                for (int k = 0; k < kCluster; ++k) { xd[k][R] = e; xd[k][R + 1] = fl0; }
                // every reader of the four flags is past the barrier above; the next writers come after the barriers below
                m.flags[0] = 0; m.flags[1] = 0; m.flags[2] = 0; m.flags[3] = 0;
            }
        }
        cluster.sync();
        // ================= gather: the same sums, in rank order, in every CTA
        float err = 0.0f;
        int fl = 0;
        {
#pragma unroll
            for (int k = 0; k < kCluster; ++k) { err += xb[k * XS + R]; fl |= __float_as_int(xb[k * XS + R + 1]); }
            for (int j = tid; j < Cn; j += kNT) {
                float c = 0.0f;
#pragma unroll
                for (int k = 0; k < kCluster; ++k) c += xb[k * XS + j];
                if (!(c > kSumLo && c < kSumHi)) m.flags[2] = 1;
                const float vn = m.dd[j] / c;
                if (!(vn > kDriftLo && vn < kDriftHi)) m.flags[3] = 1;
                vnew[j] = vn;
            }
        }
        __syncthreads();
        const bool check = a.tol > 0.0f && (t % a.check_every == 0);
        const bool bad_rows = (fl & 1) != 0;
        if (t >= a.max_iters || (check && err <= (float)tol_abs)) {
            if (bad_rows) { handed_back = true; break; }                 // the error of these rows means nothing
            err_out = (float)((double)err / sum_st);
            if (a.tol > 0.0f && !(err <= (float)tol_abs)) info |= TAOT_INFO_SINKHORN_CAP;
            break;
        }
        if (bad_rows || m.flags[2] != 0) { handed_back = true; break; }  // sums left the safe range (same in all CTAs)
        // ---- commit (u', v'); fold them into (alpha, beta) if they drifted
        const bool drift = (fl & 2) != 0 || m.flags[3] != 0;
        if (drift) {
            __syncthreads();
            for (int i = i0 + tid; i < i1; i += kNT) { m.alpha[i] += log((double)unew[i]); ucur[i] = 1.0f; unew[i] = 1.0f; }
            for (int j = tid; j < Cn; j += kNT) { m.beta[j] += log((double)vnew[j]); vcur[j] = 1.0f; vnew[j] = 1.0f; }
            __syncthreads();
            rebuild();
            __syncthreads();
        } else {
            { float* x = ucur; ucur = unew; unew = x; }
            { float* x = vcur; vcur = vnew; vnew = x; }
        }
        ++t;
    }
    if (handed_back) {
        // every CTA took this branch in the same iteration, after the barrier that completed all remote stores
        if (rank == 0 && tid == 0) a.iters[b] = kHandBack;
        return;
    }

    // ---- T = diag(u) M diag(v) from the total potentials, then the column cap
    __syncthreads();
    for (int i = i0 + tid; i < i1; i += kNT) m.alpha[i] += log((double)ucur[i]);
    for (int j = tid; j < Cn; j += kNT) m.beta[j] += log((double)vcur[j]);
    __syncthreads();
    rebuild();
    __syncthreads();
    float* xb = m.xbuf + ((t + 1) & 1) * kCluster * XS;                  // the blocks the last iteration did not use
    {
        float* xd[kCluster];
#pragma unroll
        for (int k = 0; k < kCluster; ++k) xd[k] = cluster.map_shared_rank(xb, k) + rank * XS;
        for (int j = tid; j < Cn; j += kNT) {
            float cs = 0.0f;
            for (int i = i0; i < i1; ++i) cs += m.Ks[(i - i0) * Cn + j];
#pragma unroll
            for (int k = 0; k < kCluster; ++k) xd[k][j] = cs;
        }
    }
    // zero the R x R block (shared between the CTAs) before anyone writes entries into it
    for (int64_t q = (int64_t)rank * kNT + tid; q < (int64_t)R * R; q += (int64_t)kCluster * kNT) out[q] = 0.0f;
    __threadfence();
    cluster.sync();
    for (int j = tid; j < Cn; j += kNT) {
        double cs = 0.0;
#pragma unroll
        for (int k = 0; k < kCluster; ++k) cs += (double)xb[k * XS + j];
        m.vn[j] = (float)fmin(1.0, (double)m.dd[j] / (cs + (double)a.eps0));
    }
    __syncthreads();
    int nonfinite = 0;
    {
        const int n = (i1 - i0) * Cn;
        for (int q = tid; q < n; q += kNT) {
            const int il = q / Cn, j = q - il * Cn;
            const float val = m.Ks[q] * m.vn[j];
            if (!isfinite(val)) nonfinite = 1;
            out[(int64_t)m.hot[i0 + il] * R + m.cold[j]] = val;
        }
    }
    nonfinite = __syncthreads_or(nonfinite);
    if (nonfinite && tid == 0) atomicOr(a.info + b, TAOT_INFO_NONFINITE);
    if (rank == 0 && tid == 0) {
        a.iters[b] = t;
        a.row_err[b] = err_out;
        if (info) atomicOr(a.info + b, info);
    }
}

}  // namespace

int taot_launch_sinkhorn_cluster(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st)
{
    const int R = h->p.R;
    const size_t state = (csmem_state_bytes(R) + 15) & ~(size_t)15;
    const size_t budget = 226 * 1024;                                     // the kernel also has a few static bytes
    if (state + 4096 > budget) return 0;                                 // no room for a slice: nothing launched
    const int32_t kcap = (int32_t)((budget - state) / sizeof(float));
    const size_t smem = state + sizeof(float) * (size_t)kcap;
    TAOT_CUDA_OK(cudaFuncSetAttribute(sinkhorn_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    sinkhorn_cluster_kernel<<<(unsigned)B * kCluster, kNT, smem, st>>>(a, kcap);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
