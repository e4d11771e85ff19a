// Register-tile Sinkhorn kernel, up to 64 ranks, register-capped build for large batches (20 problems per SM).
#include "sinkhorn_tile.cuh"

int taot_launch_sinkhorn_tile_r64_batch(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st)
{
    if (a.tol > 0.0f) sinkhorn_tile_kernel<1, 2, 8, 16, 32, 20, true><<<B, 32, 0, st>>>(a, (int64_t)B);
    else sinkhorn_tile_kernel<1, 2, 8, 16, 32, 20, false><<<B, 32, 0, st>>>(a, (int64_t)B);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
