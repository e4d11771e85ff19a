// Register-tile Sinkhorn kernels: the multi-warp instantiations (up to 128 / 256 ranks) and the dispatch over all
// of them.  The one-warp instantiations are compiled in translation units of their own (sinkhorn_tile_r*.cu) so
// that the build runs them in parallel.
#include "sinkhorn_tile.cuh"

int taot_launch_sinkhorn_tile_r32(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);
int taot_launch_sinkhorn_tile_r32_batch(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);
int taot_launch_sinkhorn_tile_r64(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);
int taot_launch_sinkhorn_tile_r64_batch(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);

int taot_launch_sinkhorn_tile(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st)
{
    const int R = h->p.R;
    // a batch that fills the GPU several times over is bound by how many problems an SM holds, not by the latency of
    // one: it takes the register-capped builds
    const bool batch = B >= 4 * h->sm_count;
    if (R <= 32) return batch ? taot_launch_sinkhorn_tile_r32_batch(a, B, h->sm_count, st) : taot_launch_sinkhorn_tile_r32(a, B, h->sm_count, st);
    if (R <= 64) return batch ? taot_launch_sinkhorn_tile_r64_batch(a, B, h->sm_count, st) : taot_launch_sinkhorn_tile_r64(a, B, h->sm_count, st);
    if (R <= 128) sinkhorn_tile_kernel<4, 4, 4, 8, 16, 1><<<B, 128, 0, st>>>(a, (int64_t)B);
    else sinkhorn_tile_kernel<16, 8, 2, 4, 8, 1><<<B, 512, 0, st>>>(a, (int64_t)B);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
