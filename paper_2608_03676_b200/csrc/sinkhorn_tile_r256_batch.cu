// Register-tile Sinkhorn kernel for large batches of problems with up to 256 ranks: 4 warps per problem instead of
// 16 (4 or 8 rows per warp).  Fewer warps per problem means fewer reduction, broadcast and barrier instructions
// per iteration in total, which is what a batch that fills the GPU is bound by; problems with more than 32 supply
// ranks come back marked for the 16-warp kernel.
#include "sinkhorn_tile.cuh"

int taot_launch_sinkhorn_tile_r256_batch(const SinkArgs& a, int32_t B, cudaStream_t st)
{
    sinkhorn_tile_kernel<4, 8, 4, 8, 8, 1><<<B, 128, 0, st>>>(a, (int64_t)B);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
