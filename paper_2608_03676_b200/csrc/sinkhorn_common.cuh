// Shared by the two Sinkhorn kernels (Appendix A.2): arguments, safe ranges, set-up helpers.
#pragma once

#include "taot_internal.cuh"

namespace taot_sk {

struct SinkArgs {
    const float* s;
    const float* d;
    const float* C;
    const double* rowlse0;
    float* plan;
    int32_t* iters;
    float* row_err;
    int32_t* info;
    int32_t R;
    int32_t kcap;
    double inv_eps;
    float eps0;
    int32_t max_iters;
    float tol;
    int32_t check_every;
    int32_t only_marked;     // generic kernel: solve only the problems the register-tile kernel handed back
    int32_t skip_solved;     // tile kernels: solve only the problems an earlier kernel of the chain handed back
    float* kt_global;        // [B][kcap_global] kernel-matrix scratch in global memory for problems too big for
    int64_t kcap_global;     // shared memory (floats per problem); null / 0 if the handle has none
};

// exp(x) rounded to fp32 for an fp64 argument of either sign and any magnitude the solve meets: x = xh + xl with
// xh = fl32(x), exp(x) = expf(xh) * (1 + xl).  Relative error ~3e-7 (expf is the accurate one, 2 ulp), at a small
// fraction of the cost of an fp64 exponential on this GPU.
__device__ __forceinline__ float exp_split(double x)
{
    const float xh = (float)x;
    const float xl = (float)(x - (double)xh);
    return expf(xh) * (1.0f + xl);
}

constexpr float kDriftLo = 4.2483543e-18f;  // e^-40
constexpr float kDriftHi = 2.3538527e17f;   // e^+40
constexpr float kSumLo = 1e-30f;
constexpr float kSumHi = 1e30f;
constexpr int kHandBack = -1;               // iters[b] value meaning "not solved here"

// ordered compaction of {i < R : val[i] > 0} into list[], positions into pos[]; returns the count
__device__ inline int compact_positive(const float* val, int R, int32_t* list, int32_t* pos, int32_t* wcnt)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NW = blockDim.x >> 5;
    int total = 0;
    for (int base = 0; base < R; base += blockDim.x) {
        const int i = base + tid;
        const bool p = (i < R) && (val[i] > 0.0f);
        const unsigned m = __ballot_sync(0xffffffffu, p);
        if (lane == 0) wcnt[warp] = __popc(m);
        __syncthreads();
        int off = total;
        for (int w = 0; w < warp; ++w) off += wcnt[w];
        if (i < R) pos[i] = -1;
        if (p) {
            const int q = off + __popc(m & ((1u << lane) - 1u));
            list[q] = i;
            pos[i] = q;
        }
        for (int w = 0; w < NW; ++w) total += wcnt[w];
        __syncthreads();
    }
    return total;
}

}  // namespace taot_sk
