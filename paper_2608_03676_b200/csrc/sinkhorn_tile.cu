// Phase 1 fast path: Sinkhorn-Knopp (Appendix A.2) with the absorbed kernel matrix K~ held in
// REGISTERS.  Same arithmetic as the shared-memory kernel in sinkhorn.cu (absorbed potentials,
// fp32 mat-vecs, fp64 folds), different data placement:
//
//   warp w owns compact rows [w*RPW, (w+1)*RPW)  (rows = ranks with supply),
//   lane l owns compact columns l + 32*g, g < CG (columns = ranks with demand),
//   K[a][g] in registers; every warp keeps v~ for its lane's columns in registers.
//
// Half-step 1 (row sums) is warp-local: RPW partial sums per lane are reduced across the 32 lanes
// by a transposing butterfly (RPW-1 + log2(32/RPW) shuffles for all rows together), after which
// lane a holds row a's sum and computes u~_a = s~_a / r_a.  Half-step 2 (column sums) is
// lane-local over the warp's rows (u~_a broadcast by shuffle); with several warps the partials
// meet in shared memory (two block barriers per iteration, none with one warp).
//
// A problem that does not fit the tile (more than NW*RPW rows with supply), or whose fp32 sums
// leave the safe range, is handed back (iters[b] = -1) and solved by the shared-memory kernel.
#include "sinkhorn_common.cuh"

using namespace taot_sk;

namespace {

constexpr unsigned kFull = 0xffffffffu;

// Sum over the 32 lanes of N per-lane values at once: on return the value is the total of
// p[lane & (N-1)].  N a power of two, 1 <= N <= 32.
template <int N>
__device__ __forceinline__ float transpose_reduce(float (&p)[N], int lane)
{
#pragma unroll
    for (int off = N / 2; off >= 1; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int k = 0; k < off; ++k) {
            const float send = up ? p[k] : p[k + off];
            const float keep = up ? p[k + off] : p[k];
            p[k] = keep + __shfl_xor_sync(kFull, send, off);
        }
    }
    float v = p[0];
#pragma unroll
    for (int off = N; off < 32; off <<= 1) v += __shfl_xor_sync(kFull, v, off);
    return v;
}

template <int NW, int RPW, int CG>
__global__ void __launch_bounds__(NW * 32)
sinkhorn_tile_kernel(SinkArgs a)
{
    constexpr int RMAX = 32 * CG, NT = NW * 32;
    __shared__ double sh_alpha[RMAX], sh_beta[RMAX], sh_phin[RMAX], sh_red[64];
    __shared__ float sh_st[RMAX], sh_dd[RMAX], sh_sv[RMAX], sh_dv[RMAX], sh_vs[RMAX];
    __shared__ float sh_part[NW > 1 ? NW * RMAX : 1];
    __shared__ float sh_errw[32];
    __shared__ int32_t sh_hot[RMAX], sh_cold[RMAX], sh_hpos[RMAX], sh_cpos[RMAX], sh_wcnt[32];
    __shared__ int sh_flags[4];             // [parity*2 + 0] bad sum, [parity*2 + 1] drift
    __shared__ double s_sum[2];

    const int R = a.R, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t b = blockIdx.x;

    // ---- supply scaling gamma = min(1, sum d / max(sum s, eps0)), compaction of supply / demand ranks
    {
        double ps = 0.0, pd = 0.0;
        for (int i = tid; i < R; i += NT) {
            const float sv = a.s[b * R + i], dv = a.d[b * R + i];
            ps += sv > 0.0f ? (double)sv : 0.0;
            pd += dv > 0.0f ? (double)dv : 0.0;
        }
        for (int o = 16; o > 0; o >>= 1) {
            ps += __shfl_xor_sync(kFull, ps, o);
            pd += __shfl_xor_sync(kFull, pd, o);
        }
        if (lane == 0) { sh_red[warp] = ps; sh_red[32 + warp] = pd; }
        if (tid < 4) sh_flags[tid] = 0;
        __syncthreads();
        if (tid == 0) {
            double S = 0.0, D = 0.0;
            for (int w = 0; w < NW; ++w) { S += sh_red[w]; D += sh_red[32 + w]; }
            s_sum[0] = S; s_sum[1] = D;
        }
        __syncthreads();
    }
    const double sum_s = s_sum[0], sum_d = s_sum[1];
    const double gamma = fmin(1.0, sum_d / fmax(sum_s, (double)a.eps0));
    for (int i = tid; i < R; i += NT) {
        const float sv = a.s[b * R + i], dv = a.d[b * R + i];
        sh_sv[i] = sv > 0.0f ? (float)(gamma * (double)sv) : 0.0f;
        sh_dv[i] = dv > 0.0f ? dv : 0.0f;
    }
    __syncthreads();
    const int Hn = compact_positive(sh_sv, R, sh_hot, sh_hpos, sh_wcnt);
    const int Cn = compact_positive(sh_dv, R, sh_cold, sh_cpos, sh_wcnt);
    if (Hn > NW * RPW) {                     // does not fit this tile: the other kernel takes it
        if (tid == 0) a.iters[b] = kHandBack;
        return;
    }
    for (int i = tid; i < Hn; i += NT) sh_st[i] = sh_sv[sh_hot[i]];
    for (int j = tid; j < Cn; j += NT) sh_dd[j] = sh_dv[sh_cold[j]];
    __syncthreads();

    int info = 0;
    if (sum_s > sum_d) info |= TAOT_INFO_SUPPLY_SCALED;
    float* out = a.plan + b * (int64_t)R * R;
    if (Hn == 0 || Cn == 0) {
        for (int q = tid; q < R * R; q += NT) out[q] = 0.0f;
        if (tid == 0) {
            a.iters[b] = 0;
            a.row_err[b] = 0.0f;
            if (info) atomicOr(a.info + b, info);
        }
        return;
    }
    double sum_st = 0.0;
    for (int i = 0; i < Hn; ++i) sum_st += (double)sh_st[i];          // same order in every thread
    const double tol_abs = (double)a.tol * sum_st;

    // ---- iteration 1 in the log domain (v = 1 on every rank): phi = log s~ - LSE_j(-C_ij/eps) over all j,
    //      psi_j = log d_j - LSE_i(phi_i - C_ij/eps)
    for (int i = tid; i < Hn; i += NT) sh_phin[i] = log((double)sh_st[i]) - a.rowlse0[sh_hot[i]];
    __syncthreads();
    for (int j = tid; j < Cn; j += NT) {
        const int cj = sh_cold[j];
        double mx = -INFINITY;
        for (int i = 0; i < Hn; ++i) {
            const double x = sh_phin[i] - (double)a.C[(int64_t)sh_hot[i] * R + cj] * a.inv_eps;
            mx = x > mx ? x : mx;
        }
        double acc = 0.0;
        for (int i = 0; i < Hn; ++i)
            acc += exp(sh_phin[i] - (double)a.C[(int64_t)sh_hot[i] * R + cj] * a.inv_eps - mx);
        sh_beta[j] = log((double)sh_dd[j]) - (mx + log(acc));
    }
    for (int i = tid; i < Hn; i += NT) sh_alpha[i] = sh_phin[i];
    __syncthreads();

    // ---- this thread's tile and the scalars it owns
    const int row0 = warp * RPW;
    const int rowl = row0 + (lane & (RPW - 1));       // the row whose sum this lane ends up holding
    const bool row_ok = rowl < Hn;
    const float st_l = row_ok ? sh_st[rowl] : 1.0f;
    float K[RPW][CG];
    float ddg[CG], vreg[CG];
    bool col_ok[CG];
#pragma unroll
    for (int g = 0; g < CG; ++g) {
        const int col = lane + 32 * g;
        col_ok[g] = col < Cn;
        ddg[g] = col_ok[g] ? sh_dd[col] : 1.0f;
        vreg[g] = 1.0f;
    }
    auto build_tile = [&]() {
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) {
            const int row = row0 + aa;
#pragma unroll
            for (int g = 0; g < CG; ++g) {
                const int col = lane + 32 * g;
                float v = 0.0f;
                if (row < Hn && col < Cn) {
                    const double c = (double)a.C[(int64_t)sh_hot[row] * R + sh_cold[col]] * a.inv_eps;
                    v = (float)exp(sh_alpha[row] + sh_beta[col] - c);
                }
                K[aa][g] = v;
            }
        }
    };
    build_tile();
    float uo = 1.0f;                 // committed u~ of row `rowl`
    int t = 1;
    float err_out = 0.0f;
    bool hand_back = false;

    for (;;) {
        const int par = (t & 1) * 2;
        // ================= half-step 1: r = K~ v~ (row sums of iterate t), u' = s~ / r
        float p[RPW];
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) {
            float acc = 0.0f;
#pragma unroll
            for (int g = 0; g < CG; ++g) acc = fmaf(K[aa][g], vreg[g], acc);
            p[aa] = acc;
        }
        const float r = transpose_reduce<RPW>(p, lane);
        const float un = row_ok ? st_l / r : 1.0f;
        float e = (row_ok && lane < RPW) ? fabsf(fmaf(uo, r, -st_l)) : 0.0f;
        bool bad = row_ok && !(r > kSumLo && r < kSumHi);
        bool drift = row_ok && !(un > kDriftLo && un < kDriftHi);
        for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(kFull, e, o);
        // column partials over this warp's rows, with the proposed u'
        float cp[CG];
#pragma unroll
        for (int g = 0; g < CG; ++g) cp[g] = 0.0f;
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) {
            const float ua = __shfl_sync(kFull, un, aa);
#pragma unroll
            for (int g = 0; g < CG; ++g) cp[g] = fmaf(K[aa][g], ua, cp[g]);
        }
        double err;
        if (NW == 1) {
            err = (double)e;
        } else {
#pragma unroll
            for (int g = 0; g < CG; ++g) sh_part[warp * RMAX + lane + 32 * g] = cp[g];
            if (lane == 0) sh_errw[warp] = e;
            if (bad) sh_flags[par] = 1;
            if (drift) sh_flags[par + 1] = 1;
            __syncthreads();
            err = 0.0;
            for (int w = 0; w < NW; ++w) err += (double)sh_errw[w];
            if (tid == 0) { sh_flags[(par ^ 2)] = 0; sh_flags[(par ^ 2) + 1] = 0; }
        }
        // ---- the row sums just computed belong to iterate t: stop here?
        const bool check = a.tol > 0.0f && (t % a.check_every == 0);
        if (NW == 1) bad = __any_sync(kFull, bad);
        else bad = sh_flags[par] != 0;
        if (bad) { hand_back = true; break; }
        if (t >= a.max_iters || (check && err <= tol_abs)) {
            err_out = (float)(err / sum_st);
            if (a.tol > 0.0f && !(err <= tol_abs)) info |= TAOT_INFO_SINKHORN_CAP;
            break;
        }
        // ================= half-step 2: c = K~^T u', v' = d / c
        if (NW == 1) {
            bool bad2 = false;
#pragma unroll
            for (int g = 0; g < CG; ++g) {
                const float c = cp[g];
                if (col_ok[g]) {
                    bad2 |= !(c > kSumLo && c < kSumHi);
                    const float vn = ddg[g] / c;
                    drift |= !(vn > kDriftLo && vn < kDriftHi);
                    vreg[g] = vn;
                }
            }
            if (__any_sync(kFull, bad2)) { hand_back = true; break; }
            drift = __any_sync(kFull, drift);
        } else {
            for (int j = tid; j < Cn; j += NT) {
                float c = 0.0f;
#pragma unroll
                for (int w = 0; w < NW; ++w) c += sh_part[w * RMAX + j];
                if (!(c > kSumLo && c < kSumHi)) sh_flags[par] = 1;
                const float vn = sh_dd[j] / c;
                if (!(vn > kDriftLo && vn < kDriftHi)) sh_flags[par + 1] = 1;
                sh_vs[j] = vn;
            }
            __syncthreads();
            if (sh_flags[par]) { hand_back = true; break; }
            drift = sh_flags[par + 1] != 0;
#pragma unroll
            for (int g = 0; g < CG; ++g) vreg[g] = col_ok[g] ? sh_vs[lane + 32 * g] : 1.0f;
        }
        uo = un;
        ++t;
        if (drift) {
            // fold u~, v~ into the fp64 potentials and rebuild the tile around them
            if (row_ok && lane < RPW) sh_alpha[rowl] += log((double)uo);
            if (NW == 1) {
#pragma unroll
                for (int g = 0; g < CG; ++g)
                    if (col_ok[g]) sh_beta[lane + 32 * g] += log((double)vreg[g]);
                __syncwarp();
            } else {
                for (int j = tid; j < Cn; j += NT) sh_beta[j] += log((double)sh_vs[j]);
                __syncthreads();
            }
            uo = 1.0f;
#pragma unroll
            for (int g = 0; g < CG; ++g) vreg[g] = 1.0f;
            build_tile();
            if (NW > 1) __syncthreads();
        }
    }

    if (hand_back) {
        if (tid == 0) a.iters[b] = kHandBack;
        return;
    }

    // ---- T = diag(u) M diag(v) from the total potentials, then the column cap
    if (NW > 1) __syncthreads();
    if (row_ok && lane < RPW) sh_alpha[rowl] += log((double)uo);
    if (warp == 0 || NW == 1) {
#pragma unroll
        for (int g = 0; g < CG; ++g)
            if (col_ok[g]) sh_beta[lane + 32 * g] += log((double)vreg[g]);     // every warp holds the same v~
    }
    __syncthreads();
    build_tile();
    float cs[CG];
#pragma unroll
    for (int g = 0; g < CG; ++g) {
        float acc = 0.0f;
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) acc += K[aa][g];
        cs[g] = acc;
    }
    float fg[CG];
    if (NW == 1) {
#pragma unroll
        for (int g = 0; g < CG; ++g)
            fg[g] = col_ok[g] ? (float)fmin(1.0, (double)ddg[g] / ((double)cs[g] + (double)a.eps0)) : 0.0f;
    } else {
#pragma unroll
        for (int g = 0; g < CG; ++g) sh_part[warp * RMAX + lane + 32 * g] = cs[g];
        __syncthreads();
        for (int j = tid; j < Cn; j += NT) {
            double c = 0.0;
#pragma unroll
            for (int w = 0; w < NW; ++w) c += (double)sh_part[w * RMAX + j];
            sh_vs[j] = (float)fmin(1.0, (double)sh_dd[j] / (c + (double)a.eps0));
        }
        __syncthreads();
#pragma unroll
        for (int g = 0; g < CG; ++g) fg[g] = col_ok[g] ? sh_vs[lane + 32 * g] : 0.0f;
    }
    // zero the R x R block, then scatter the hot x cold entries
    for (int q = tid; q < R * R; q += NT) out[q] = 0.0f;
    __syncthreads();
    int nonfinite = 0;
#pragma unroll
    for (int aa = 0; aa < RPW; ++aa) {
        const int row = row0 + aa;
        if (row >= Hn) continue;
        float* orow = out + (int64_t)sh_hot[row] * R;
#pragma unroll
        for (int g = 0; g < CG; ++g) {
            if (!col_ok[g]) continue;
            const float val = K[aa][g] * fg[g];
            if (!isfinite(val)) nonfinite = 1;
            orow[sh_cold[lane + 32 * g]] = val;
        }
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

int taot_launch_sinkhorn_tile(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st)
{
    const int R = h->p.R;
    if (R <= 32) sinkhorn_tile_kernel<1, 16, 1><<<B, 32, 0, st>>>(a);
    else if (R <= 64) sinkhorn_tile_kernel<1, 32, 2><<<B, 32, 0, st>>>(a);
    else if (R <= 128) sinkhorn_tile_kernel<4, 16, 4><<<B, 128, 0, st>>>(a);
    else sinkhorn_tile_kernel<16, 8, 8><<<B, 512, 0, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
