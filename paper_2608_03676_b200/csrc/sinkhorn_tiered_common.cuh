// Shared by the two tier-by-tier Sinkhorn kernels (sinkhorn_tiered.cu: one warp per problem; sinkhorn_tiered_mw.cu:
// eight warps per problem): the tier costs, the first iteration's column potential in the log domain, and the rows of
// the final plan.  The factorisation of the sums itself is described at the top of sinkhorn_tiered.cu.
#pragma once

#include "sinkhorn_common.cuh"

namespace taot_sk {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float rcp_fast(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float exp_or_zero(double x) { return x == -INFINITY ? 0.0f : exp_split(x); }

struct TierCosts {
    double c1, c2, c3;            // cost / eps of the three tiers off the diagonal
};

// C_ij / eps for i != j, from the indices alone: kNode ranks per node, kGroup ranks per rail group
template <int kNode, int kGroup>
__device__ __forceinline__ double tier_cost(const TierCosts& tc, int i, int j)
{
    return (i / kNode == j / kNode) ? tc.c1 : ((i / kGroup == j / kGroup) ? tc.c2 : tc.c3);
}

// Iteration 1, second half, in the log domain (Appendix A.2 with v = 1 on every rank in the first half):
// psi_q = log d_q - LSE_i(phi_i - C_iq/eps) over the Hn supply ranks hot[], phi = alpha.
template <int kNode, int kGroup>
__device__ __forceinline__ double first_column_potential(const TierCosts& tc, const double* alpha, const int32_t* hot, int Hn,
                                                         int q, float dq)
{
    double mx = -INFINITY;
    for (int h = 0; h < Hn; ++h) {
        const int r = hot[h];
        const double v = alpha[r] - tier_cost<kNode, kGroup>(tc, r, q);
        mx = v > mx ? v : mx;
    }
    double acc = 0.0;
    for (int h = 0; h < Hn; ++h) {
        const int r = hot[h];
        acc += (double)exp_split(alpha[r] - tier_cost<kNode, kGroup>(tc, r, q) - mx);
    }
    return log((double)dq) - (mx + log(acc));
}

// Rows row0, row0 + step, ... of the final plan T_ij = exp(alpha_i + beta_j - C_ij/eps) * cap_j by one warp (lane =
// column modulo 32); cap[] is 0 off the demand ranks.  Returns 1 if a value came out non-finite.
template <int kNode, int kGroup>
__device__ __forceinline__ int write_plan_rows(const TierCosts& tc, const double* alpha, const double* beta, const float* cap,
                                               int R, int row0, int step, int lane, float* out)
{
    int nonfinite = 0;
    for (int row = row0; row < R; row += step) {
        const double al = alpha[row];
        float* orow = out + (int64_t)row * R;
        if (al == -INFINITY) {
            for (int j = lane; j < R; j += 32) orow[j] = 0.0f;
            continue;
        }
#pragma unroll 4
        for (int j = lane; j < R; j += 32) {
            const float fg = cap[j];
            float val = 0.0f;
            if (fg > 0.0f) {
                val = exp_split(al + beta[j] - tier_cost<kNode, kGroup>(tc, row, j)) * fg;
                if (!isfinite(val)) nonfinite = 1;
            }
            orow[j] = val;
        }
    }
    return nonfinite;
}

}  // namespace taot_sk
