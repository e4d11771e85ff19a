// Register-tile Sinkhorn kernels: the multi-warp instantiations (up to 128 / 256 ranks) and the dispatch over all
// of them.  The one-warp instantiations are compiled in translation units of their own (sinkhorn_tile_r*.cu) so
// that the build runs them in parallel.
#include "sinkhorn_tile.cuh"

int taot_launch_sinkhorn_tile_r32(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);
int taot_launch_sinkhorn_tile_r32_batch(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);
int taot_launch_sinkhorn_tile_r64(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);
int taot_launch_sinkhorn_tile_r64_batch(const SinkArgs& a, int32_t B, int sm_count, cudaStream_t st);

int taot_launch_sinkhorn_tile_r256_batch(const SinkArgs& a, int32_t B, cudaStream_t st);

int taot_launch_sinkhorn_tile(taot_handle_t h, const SinkArgs& a_in, int32_t B, cudaStream_t st)
{
    SinkArgs a = a_in;
    a.skip_solved = 0;
    const int R = h->p.R;
    // a batch that fills the GPU several times over is bound by how many problems an SM holds, not by the latency of
    // one: it takes the register-capped builds
    const bool batch = B >= 4 * h->sm_count;
    if (R <= 32) return batch ? taot_launch_sinkhorn_tile_r32_batch(a, B, h->sm_count, st) : taot_launch_sinkhorn_tile_r32(a, B, h->sm_count, st);
    if (R <= 64) return batch ? taot_launch_sinkhorn_tile_r64_batch(a, B, h->sm_count, st) : taot_launch_sinkhorn_tile_r64(a, B, h->sm_count, st);
    int launched = 1;
    if (batch) {
        // 4 warps per problem first; problems with more than 32 supply ranks come back marked for the kernels below
        const int n = taot_launch_sinkhorn_tile_r256_batch(a, B, st);
        if (n < 0) return n;
        launched += n;
        a.skip_solved = 1;
    }
    if (R <= 128) sinkhorn_tile_kernel<4, 4, 4, 8, 16, 1><<<B, 128, 0, st>>>(a, (int64_t)B);
    else sinkhorn_tile_kernel<16, 8, 2, 4, 8, 1><<<B, 512, 0, st>>>(a, (int64_t)B);
    TAOT_CUDA_OK(cudaGetLastError());
    return launched;
}
