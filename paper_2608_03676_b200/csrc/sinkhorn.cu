// Phase 1: batched entropic optimal transport by Sinkhorn-Knopp (Appendix A.2).
//
// One CTA per problem.  The paper's iteration u = s~/(M v), v = d/(M^T u) is carried in the
// "absorbed" form: total log-potentials are split as  log u = alpha + log u~,  log v = beta +
// log v~  with (alpha, beta) in fp64 and (u~, v~) in fp32 near 1, and the kernel matrix held on
// chip is  K~_ij = exp(alpha_i + beta_j - C_ij/eps)  rounded to fp32.  A half-step is then an
// fp32 mat-vec over K~ followed by a divide, exactly the paper's GEMV form, but it cannot
// under- or overflow for any C/eps: whenever u~ or v~ drifts outside [e^-40, e^40] the factors
// are folded into (alpha, beta) and K~ is rebuilt (fp64 exp, a few times per solve).  Only rows
// with supply and columns with demand carry flow, so K~ is compacted to |hot| x |cold|.
// The first iteration (v = 1 on every rank) is done in the log domain in fp64; so is any
// iteration whose fp32 sums leave the safe range, which makes the solve total.
//
// Stopping: half-step 1 of iteration t+1 produces the row sums of iterate t for free
// (rowsum_i = u~_i * (K~ v~)_i), so the tolerance test costs nothing extra.
#include "sinkhorn_common.cuh"

using namespace taot_sk;

namespace {

struct Smem {
    double* alpha;   // [R] by compact hot index
    double* beta;    // [R] by compact cold index
    double* phin;    // [R] scratch: new log-potential of the rows (slow path)
    double* errp;    // [32]
    float* st;       // [R] scaled supply, compact
    float* dd;       // [R] demand, compact
    float* u;        // [R]
    float* un;       // [R]
    float* v;        // [R]
    float* vn;       // [R]
    float* part;     // [max(NT, R)]
    int32_t* hot;    // [R] compact -> rank
    int32_t* cold;   // [R]
    int32_t* hpos;   // [R] rank -> compact or -1
    int32_t* cpos;   // [R]
    int32_t* wcnt;   // [32]
    int32_t* flags;  // [4]: 0 bad sum, 1 drift
    float* Kt;       // [kcap]
};

__device__ __forceinline__ Smem carve(unsigned char* base, int R, int NT)
{
    Smem m;
    double* dp = reinterpret_cast<double*>(base);
    m.alpha = dp; dp += R;
    m.beta = dp; dp += R;
    m.phin = dp; dp += R;
    m.errp = dp; dp += 32;
    float* fp = reinterpret_cast<float*>(dp);
    m.st = fp; fp += R;
    m.dd = fp; fp += R;
    m.u = fp; fp += R;
    m.un = fp; fp += R;
    m.v = fp; fp += R;
    m.vn = fp; fp += R;
    m.part = fp; fp += (NT > R ? NT : R);
    int32_t* ip = reinterpret_cast<int32_t*>(fp);
    m.hot = ip; ip += R;
    m.cold = ip; ip += R;
    m.hpos = ip; ip += R;
    m.cpos = ip; ip += R;
    m.wcnt = ip; ip += 32;
    m.flags = ip; ip += 4;
    m.Kt = reinterpret_cast<float*>(ip);
    return m;
}

size_t smem_bytes(int R, int NT, int kcap)
{
    return sizeof(double) * (3 * R + 32) + sizeof(float) * (6 * R + (NT > R ? NT : R)) +
           sizeof(int32_t) * (4 * R + 36) + sizeof(float) * (size_t)kcap;
}

// K~_ij = exp(alpha_i + beta_j - C_ij/eps), fp64 exponent and exp, rounded once to fp32
__device__ void rebuild_kernel(const Smem& m, const SinkArgs& a, int Hn, int Cn)
{
    for (int q = threadIdx.x; q < Hn * Cn; q += blockDim.x) {
        const int i = q / Cn, j = q - i * Cn;
        const double c = (double)a.C[(int64_t)m.hot[i] * a.R + m.cold[j]] * a.inv_eps;
        m.Kt[q] = (float)exp(m.alpha[i] + m.beta[j] - c);
    }
}

// slow path, rows: L_i = LSE_j(psi_j - C_ij/eps) with psi = beta + log v~;  phin_i = log s~_i - L_i;
// contributes |exp(phi_i + L_i) - s~_i| to the row violation (phi = alpha + log u~).
__device__ void slow_half1(const Smem& m, const SinkArgs& a, int Hn, int Cn)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double e = 0.0;
    for (int i = tid; i < Hn; i += blockDim.x) {
        const float* crow = a.C + (int64_t)m.hot[i] * a.R;
        double mx = -INFINITY;
        for (int j = 0; j < Cn; ++j) {
            const double x = m.beta[j] + log((double)m.v[j]) - (double)crow[m.cold[j]] * a.inv_eps;
            mx = x > mx ? x : mx;
        }
        double acc = 0.0;
        for (int j = 0; j < Cn; ++j) {
            const double x = m.beta[j] + log((double)m.v[j]) - (double)crow[m.cold[j]] * a.inv_eps;
            acc += exp(x - mx);
        }
        const double L = mx + log(acc);
        const double phi = m.alpha[i] + log((double)m.u[i]);
        e += fabs(exp(phi + L) - (double)m.st[i]);
        m.phin[i] = log((double)m.st[i]) - L;
    }
    for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
    if (lane == 0) m.errp[warp] = e;
}

// slow path, columns: beta_j = log d_j - LSE_i(phin_i - C_ij/eps); then alpha = phin, u~ = v~ = 1
__device__ void slow_half2(const Smem& m, const SinkArgs& a, int Hn, int Cn)
{
    for (int j = threadIdx.x; j < Cn; j += blockDim.x) {
        const int cj = m.cold[j];
        double mx = -INFINITY;
        for (int i = 0; i < Hn; ++i) {
            const double x = m.phin[i] - (double)a.C[(int64_t)m.hot[i] * a.R + cj] * a.inv_eps;
            mx = x > mx ? x : mx;
        }
        double acc = 0.0;
        for (int i = 0; i < Hn; ++i) {
            const double x = m.phin[i] - (double)a.C[(int64_t)m.hot[i] * a.R + cj] * a.inv_eps;
            acc += exp(x - mx);
        }
        m.beta[j] = log((double)m.dd[j]) - (mx + log(acc));
        m.v[j] = 1.0f;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < Hn; i += blockDim.x) { m.alpha[i] = m.phin[i]; m.u[i] = 1.0f; }
    __syncthreads();
    rebuild_kernel(m, a, Hn, Cn);
    __syncthreads();
}

__global__ void __launch_bounds__(1024) sinkhorn_kernel(SinkArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int R = a.R, NT = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NW = NT >> 5;
    Smem m = carve(smem_raw, R, NT);
    const int64_t b = blockIdx.x;
    __shared__ double s_sum[2];
    if (a.only_marked && a.iters[b] != kHandBack) return;

    // ---- supply scaling gamma = min(1, sum d / max(sum s, eps0)), compaction
    if (tid == 0) { s_sum[0] = 0.0; s_sum[1] = 0.0; }
    __syncthreads();
    {
        double ps = 0.0, pd = 0.0;
        for (int i = tid; i < R; i += NT) {
            const float sv = a.s[b * R + i], dv = a.d[b * R + i];
            ps += sv > 0.0f ? (double)sv : 0.0;
            pd += dv > 0.0f ? (double)dv : 0.0;
        }
        for (int o = 16; o > 0; o >>= 1) {
            ps += __shfl_xor_sync(0xffffffffu, ps, o);
            pd += __shfl_xor_sync(0xffffffffu, pd, o);
        }
        if (lane == 0) { m.errp[warp] = ps; m.phin[warp] = pd; }   // phin is free here
        __syncthreads();
        if (tid == 0) {
            double S = 0.0, D = 0.0;
            for (int w = 0; w < NW; ++w) { S += m.errp[w]; D += m.phin[w]; }
            s_sum[0] = S; s_sum[1] = D;
        }
        __syncthreads();
    }
    const double sum_s = s_sum[0], sum_d = s_sum[1];
    const double gamma = fmin(1.0, sum_d / fmax(sum_s, (double)a.eps0));
    // scaled supply and demand by rank, in un[] / vn[] for the compaction
    for (int i = tid; i < R; i += NT) {
        const float sv = a.s[b * R + i], dv = a.d[b * R + i];
        m.un[i] = sv > 0.0f ? (float)(gamma * (double)sv) : 0.0f;
        m.vn[i] = dv > 0.0f ? dv : 0.0f;
    }
    __syncthreads();
    const int Hn = compact_positive(m.un, R, m.hot, m.hpos, m.wcnt);
    const int Cn = compact_positive(m.vn, R, m.cold, m.cpos, m.wcnt);
    for (int i = tid; i < Hn; i += NT) m.st[i] = m.un[m.hot[i]];
    for (int j = tid; j < Cn; j += NT) m.dd[j] = m.vn[m.cold[j]];
    __syncthreads();

    int info = 0;
    if (sum_s > sum_d) info |= TAOT_INFO_SUPPLY_SCALED;
    const bool empty = (Hn == 0) || (Cn == 0);
    bool too_big = (int64_t)Hn * Cn > (int64_t)a.kcap;
    if (too_big && a.kt_global != nullptr && (int64_t)Hn * Cn <= a.kcap_global) {
        m.Kt = a.kt_global + b * a.kcap_global;           // kernel matrix in global memory (L2 when the batch is small)
        too_big = false;
    }
    if (too_big) info |= TAOT_INFO_SINKHORN_SIZE;

    int t = 0;
    float err_out = 0.0f;
    if (!empty && !too_big) {
        double sum_st = 0.0;
        for (int i = 0; i < Hn; ++i) sum_st += (double)m.st[i];      // same order in every thread
        const double tol_abs = (double)a.tol * sum_st;

        // ---- iteration 1 in the log domain: v = 1 on EVERY rank, so the row normaliser is the
        //      precomputed LSE_j(-C_ij/eps) over all j
        for (int i = tid; i < Hn; i += NT) {
            m.phin[i] = log((double)m.st[i]) - a.rowlse0[m.hot[i]];
            m.u[i] = 1.0f;
        }
        __syncthreads();
        slow_half2(m, a, Hn, Cn);
        t = 1;

        // half-step-2 thread layout: G row groups x Cnp columns
        const int Cnp = (Cn + 31) & ~31;
        const int G = NT >= Cnp ? NT / Cnp : 1;
        const int cstride = NT >= Cnp ? Cnp : NT;
        const int g = tid / cstride, j0 = tid - g * cstride;

        for (;;) {
            // ================= half-step 1: r = K~ v~ ; rows of iterate t; u' = s~ / r
            if (tid < 4) m.flags[tid] = 0;
            __syncthreads();
            {
                double e = 0.0;
                for (int i = warp; i < Hn; i += NW) {
                    const float* krow = m.Kt + i * Cn;
                    float p = 0.0f;
                    for (int j = lane; j < Cn; j += 32) p = fmaf(krow[j], m.v[j], p);
                    for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
                    if (lane == 0) {
                        if (!(p > kSumLo && p < kSumHi)) m.flags[0] = 1;
                        const float un = m.st[i] / p;
                        if (!(un > kDriftLo && un < kDriftHi)) m.flags[1] = 1;
                        m.un[i] = un;
                        e += (double)fabsf(fmaf(m.u[i], p, -m.st[i]));
                    }
                }
                if (lane == 0) m.errp[warp] = e;
            }
            __syncthreads();
            bool slow = m.flags[0] != 0;
            if (slow) {                    // redo the rows exactly, from the iterate that is still intact
                __syncthreads();
                slow_half1(m, a, Hn, Cn);
                __syncthreads();
            }
            double err = 0.0;
            for (int w = 0; w < NW; ++w) err += m.errp[w];
            const bool check = a.tol > 0.0f && (t % a.check_every == 0);
            if (t >= a.max_iters || (check && err <= tol_abs)) {
                err_out = (float)(err / sum_st);
                if (a.tol > 0.0f && !(err <= tol_abs)) info |= TAOT_INFO_SINKHORN_CAP;
                break;
            }
            // ================= half-step 2: c = K~^T u' ; v' = d / c
            if (!slow) {
                for (int j = j0; j < Cn && g < G; j += cstride) {
                    float p = 0.0f;
                    for (int i = g; i < Hn; i += G) p = fmaf(m.Kt[i * Cn + j], m.un[i], p);
                    m.part[g * Cn + j] = p;
                }
                __syncthreads();
                for (int j = tid; j < Cn; j += NT) {
                    float c = 0.0f;
                    for (int gg = 0; gg < G; ++gg) c += m.part[gg * Cn + j];
                    if (!(c > kSumLo && c < kSumHi)) m.flags[0] = 1;
                    const float vn = m.dd[j] / c;
                    if (!(vn > kDriftLo && vn < kDriftHi)) m.flags[1] = 1;
                    m.vn[j] = vn;
                }
                __syncthreads();
                if (m.flags[0]) {          // columns left the safe range: finish this iteration exactly
                    slow = true;
                    for (int i = tid; i < Hn; i += NT) m.phin[i] = m.alpha[i] + log((double)m.un[i]);
                    __syncthreads();
                }
            }
            if (slow) {
                slow_half2(m, a, Hn, Cn);
            } else {
                // commit (u', v'); fold them into (alpha, beta) if they drifted
                const bool drift = m.flags[1] != 0;
                __syncthreads();
                if (drift) {
                    for (int i = tid; i < Hn; i += NT) { m.alpha[i] += log((double)m.un[i]); m.u[i] = 1.0f; }
                    for (int j = tid; j < Cn; j += NT) { m.beta[j] += log((double)m.vn[j]); m.v[j] = 1.0f; }
                    __syncthreads();
                    rebuild_kernel(m, a, Hn, Cn);
                } else {
                    for (int i = tid; i < Hn; i += NT) m.u[i] = m.un[i];
                    for (int j = tid; j < Cn; j += NT) m.v[j] = m.vn[j];
                }
                __syncthreads();
            }
            ++t;
        }

        // ---- T = diag(u) M diag(v) from the total potentials, then the column cap
        __syncthreads();
        for (int i = tid; i < Hn; i += NT) m.alpha[i] += log((double)m.u[i]);
        for (int j = tid; j < Cn; j += NT) m.beta[j] += log((double)m.v[j]);
        __syncthreads();
        rebuild_kernel(m, a, Hn, Cn);
        __syncthreads();
        for (int j = tid; j < Cn; j += NT) {
            double cs = 0.0;
            for (int i = 0; i < Hn; ++i) cs += (double)m.Kt[i * Cn + j];
            m.vn[j] = (float)fmin(1.0, (double)m.dd[j] / (cs + (double)a.eps0));
        }
        __syncthreads();
    }

    // ---- write the full R x R plan (zeros off the hot x cold block)
    int nonfinite = 0;
    float* out = a.plan + b * (int64_t)R * R;
    for (int q = tid; q < R * R; q += NT) {
        const int i = q / R, j = q - i * R;
        float val = 0.0f;
        if (!empty && !too_big) {
            const int hp = m.hpos[i], cp = m.cpos[j];
            if (hp >= 0 && cp >= 0) val = m.Kt[hp * Cn + cp] * m.vn[cp];
        }
        if (!isfinite(val)) nonfinite = 1;
        out[q] = val;
    }
    nonfinite = __syncthreads_or(nonfinite);
    if (nonfinite) info |= TAOT_INFO_NONFINITE;
    if (tid == 0) {
        a.iters[b] = t;
        a.row_err[b] = err_out;
        if (info) atomicOr(a.info + b, info);
    }
}

}  // namespace

int taot_launch_sinkhorn_tile(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st);
int taot_launch_sinkhorn_cluster(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st);
int taot_launch_sinkhorn_tiered(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st);
int taot_launch_sinkhorn_dense_tc(taot_handle_t h, const SinkArgs& a, int32_t B, float* ws_tc, cudaStream_t st);

// Caller-supplied supply / demand vectors (the stand-alone entry point; inside taot_plan they come from integer
// loads and are always finite): a problem whose s or d holds a NaN or an infinity has no solution.  One warp per
// problem rereads the inputs after the solve; for such a problem it clears the plan, reports 0 iterations and sets
// TAOT_INFO_NONFINITE.  The solve kernels themselves never index with a value derived from s or d and all their
// loops are bounded, so whatever they computed on that problem before is harmless and is overwritten here.
__global__ void __launch_bounds__(128)
sinkhorn_input_guard_kernel(const float* __restrict__ s, const float* __restrict__ d, int32_t B, int32_t R,
                            float* plan, int32_t* iters, float* row_err, int32_t* info)
{
    const int lane = threadIdx.x & 31;
    const int64_t b = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= B) return;
    bool bad = false;
    for (int r = lane; r < R; r += 32) bad |= !isfinite(s[b * R + r]) || !isfinite(d[b * R + r]);
    if (!__any_sync(0xffffffffu, bad)) return;
    float* out = plan + b * (int64_t)R * R;
    for (int64_t q = lane; q < (int64_t)R * R; q += 32) out[q] = 0.0f;
    if (lane == 0) {
        iters[b] = 0;
        row_err[b] = 0.0f;
        atomicOr(info + b, TAOT_INFO_NONFINITE);
    }
}

int taot_launch_sinkhorn_guard(taot_handle_t h, const float* d_s, const float* d_d, int32_t B, float* d_plan,
                               int32_t* d_iters, float* d_row_err, int32_t* d_info, cudaStream_t st)
{
    sinkhorn_input_guard_kernel<<<(B + 3) / 4, 128, 0, st>>>(d_s, d_d, B, h->p.R, d_plan, d_iters, d_row_err, d_info);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

int taot_launch_sinkhorn(taot_handle_t h, const float* d_s, const float* d_d, int32_t B, float* d_plan,
                         int32_t* d_iters, float* d_row_err, int32_t* d_info, float* d_kt, cudaStream_t st, float* d_tc)
{
    const taot_params& p = h->p;
    SinkArgs a;
    a.C = h->d_C; a.rowlse0 = h->d_rowlse0;
    a.R = p.R; a.kcap = h->kcap;
    a.inv_eps = 1.0 / (double)p.eps;
    a.eps0 = p.eps0; a.max_iters = p.max_iters; a.tol = p.tol;
    a.check_every = p.check_every < 1 ? 1 : p.check_every;
    a.skip_solved = 0;
    a.kt_global = h->kcap_global > 0 ? d_kt : nullptr;
    a.kcap_global = h->kcap_global;
    const int NT = p.R <= 32 ? 32 : (p.R <= 64 ? 128 : (p.R <= 128 ? 256 : (p.R <= 256 ? 512 : 1024)));
    const size_t smem = smem_bytes(p.R, NT, h->kcap);
    TAOT_CUDA_OK(cudaFuncSetAttribute(sinkhorn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int launched = 0;
    // the global scratch (if any) holds p.L problems: larger batches go through in slices
    const int32_t slice = a.kt_global ? p.L : B;
    for (int32_t b0 = 0; b0 < B; b0 += slice) {
        const int32_t nb = (B - b0) < slice ? (B - b0) : slice;
        a.s = d_s + (int64_t)b0 * p.R; a.d = d_d + (int64_t)b0 * p.R;
        a.plan = d_plan + (int64_t)b0 * p.R * p.R; a.iters = d_iters + b0; a.row_err = d_row_err + b0;
        a.info = d_info + b0;
        const int nt = taot_launch_sinkhorn_tiered(h, a, nb, st);
        if (nt < 0) return nt;
        if (nt > 0) {
            // tiered cost: O(R) sums per half-step, one warp per problem; what it hands back goes to the kernel below
            launched += nt;
            a.only_marked = 1;
        } else if (p.R <= 256) {
            // fast path: kernel matrix in registers; problems it cannot hold (or whose fp32 sums leave the
            // safe range) come back marked and are solved by the shared-memory kernel below
            a.only_marked = 1;
            const int n = taot_launch_sinkhorn_tile(h, a, nb, st);
            if (n < 0) return n;
            launched += n;
        } else {
            // beyond 256 ranks, a large batch with a fixed iteration count and a Gibbs kernel inside fp32: the whole
            // batch as dense products on the tensor cores (complete: nothing is handed on)
            const int ntc = taot_launch_sinkhorn_dense_tc(h, a, nb, d_tc, st);
            if (ntc < 0) return ntc;
            if (ntc > 0) { launched += ntc; continue; }
            // otherwise four-CTA clusters hold the kernel matrix in distributed shared memory; what they hand
            // back (or everything, if no slice fits) goes to the kernel below with the matrix in workspace
            const int n = taot_launch_sinkhorn_cluster(h, a, nb, st);
            if (n < 0) return n;
            launched += n;
            a.only_marked = n > 0 ? 1 : 0;
        }
        sinkhorn_kernel<<<nb, NT, smem, st>>>(a);
        TAOT_CUDA_OK(cudaGetLastError());
        launched += 1;
    }
    return launched;
}
