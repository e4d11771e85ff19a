// Measured arithmetic ceilings of the GPU the library runs on, for the roofline of the Sinkhorn stage: FP32
// fused multiply-add throughput and special-function (ex2) throughput.  Both kernels are pure register
// chains with enough independent accumulators per thread to cover the pipeline latency at full occupancy;
// the result is written once so that nothing is optimised away.  Not a step of the method.
#include "taot_internal.cuh"

namespace {

constexpr int kPeakThreads = 256;
constexpr int kChains = 8;
constexpr int kInner = 512;

__global__ void __launch_bounds__(kPeakThreads)
fma_peak_kernel(float* sink, int outer, float a, float b)
{
    float acc[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc[c] = (float)(threadIdx.x + c) * 1e-3f;
    for (int o = 0; o < outer; ++o) {
#pragma unroll 8
        for (int i = 0; i < kInner; ++i) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) acc[c] = fmaf(acc[c], a, b);
        }
    }
    float s = 0.0f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += acc[c];
    if (s == 12345.678f) sink[blockIdx.x * kPeakThreads + threadIdx.x] = s;      // practically never true
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(kPeakThreads)
ex2_peak_kernel(float* sink, int outer)
{
    float acc[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc[c] = (float)(threadIdx.x + c) * 1e-3f;
    for (int o = 0; o < outer; ++o) {
#pragma unroll 8
        for (int i = 0; i < kInner; ++i) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) acc[c] = ex2_approx(acc[c]) - 1.0f;   // stays in [0, 1]
        }
    }
    float s = 0.0f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += acc[c];
    if (s == 12345.678f) sink[blockIdx.x * kPeakThreads + threadIdx.x] = s;
}

// Latency of the dependent operations a one-warp Sinkhorn iteration is made of, in SM clock cycles per operation:
// one level of a shuffle reduction (shfl.xor + add), one fused multiply-add, one scaling update (rcp.approx + mul).
// One warp, one long dependent chain per measurement, timed with the SM's own cycle counter.
__global__ void __launch_bounds__(32)
latency_kernel(float* out, int n, float a, float b)
{
    const unsigned full = 0xffffffffu;
    float x = 1.0f + (float)threadIdx.x * 1e-3f;
    float res[3];
    for (int which = 0; which < 3; ++which) {
        float y = x;
        for (int pass = 0; pass < 2; ++pass) {                   // the first pass warms the instruction cache
            const long long t0 = clock64();
            if (which == 0) {
#pragma unroll 16
                for (int i = 0; i < n; ++i) y = y * 0.5f + __shfl_xor_sync(full, y, 1 << (i & 3)) * 0.5f;
            } else if (which == 1) {
#pragma unroll 16
                for (int i = 0; i < n; ++i) y = fmaf(y, a, b);
            } else {
#pragma unroll 16
                for (int i = 0; i < n; ++i) {
                    float r;
                    asm volatile("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y));
                    y = a * r + 1.0f;
                }
            }
            const long long t1 = clock64();
            res[which] = (float)(t1 - t0) / (float)n;
        }
        x += y * 1e-30f;
    }
    // level 0 carries one multiply more than a plain reduction level (it keeps the value bounded): take it off
    if (threadIdx.x == 0) {
        out[0] = res[0] - res[1];
        out[1] = res[1];
        out[2] = res[2];
        out[3] = x;
    }
}


// Latencies of the operations an auction round is a chain of, in SM clock cycles, measured the way the matching kernel
// uses them: one CTA of eight warps on an SM of its own.  [0] a dependent shared-memory load (pointer chase);
// [1] a shared-memory atomicMax whose result the next one depends on; [2] a named barrier over the eight warps, back to
// back; [3] the arbitration triple as a unit: atomicMax into a word, barrier, read-back of the word.
__global__ void __launch_bounds__(256)
round_latency_kernel(float* out, int n)
{
    __shared__ int chase[256];
    __shared__ unsigned arb[256];
    const int tid = threadIdx.x;
    chase[tid] = (tid * 37 + 11) & 255;                      // a permutation of 0..255 (37 is odd)
    arb[tid] = 0u;
    __syncthreads();
    float res[4];
    int p = tid;
    unsigned v = (unsigned)tid + 1u;
    for (int pass = 0; pass < 2; ++pass) {                   // the first pass warms the instruction cache
        long long t0 = clock64();
#pragma unroll 16
        for (int i = 0; i < n; ++i) p = chase[p];
        long long t1 = clock64();
        res[0] = (float)(t1 - t0) / (float)n;
        t0 = clock64();
#pragma unroll 16
        for (int i = 0; i < n; ++i) v = atomicMax(&arb[(tid + v) & 255], v + (unsigned)i) + 1u;
        t1 = clock64();
        res[1] = (float)(t1 - t0) / (float)n;
        t0 = clock64();
#pragma unroll 16
        for (int i = 0; i < n; ++i) asm volatile("bar.sync 1, 256;" ::: "memory");
        t1 = clock64();
        res[2] = (float)(t1 - t0) / (float)n;
        t0 = clock64();
#pragma unroll 4
        for (int i = 0; i < n; ++i) {
            atomicMax(&arb[(p + i) & 255], v + (unsigned)i);
            asm volatile("bar.sync 1, 256;" ::: "memory");
            v += arb[(p + i) & 255] & 1u;
        }
        t1 = clock64();
        res[3] = (float)(t1 - t0) / (float)n;
    }
    if (tid == 0) {
        out[0] = res[0]; out[1] = res[1]; out[2] = res[2]; out[3] = res[3];
        out[4] = (float)(p + (int)v) * 1e-30f;
    }
}

}  // namespace

extern "C" int taot_measure_latencies(float* h_cycles, void* d_sink, void* stream)
{
    if (!h_cycles || !d_sink) return TAOT_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    latency_kernel<<<1, 32, 0, st>>>(static_cast<float*>(d_sink), 4096, 0.999f, 1e-3f);
    TAOT_CUDA_OK(cudaGetLastError());
    float h[4];
    TAOT_CUDA_OK(cudaMemcpyAsync(h, d_sink, sizeof(h), cudaMemcpyDeviceToHost, st));
    TAOT_CUDA_OK(cudaStreamSynchronize(st));
    h_cycles[0] = h[0]; h_cycles[1] = h[1]; h_cycles[2] = h[2];
    return TAOT_OK;
}

extern "C" int taot_measure_alu_peaks(float* h_fma_tflops, float* h_ex2_tops, void* d_sink, void* stream)
{
    if (!h_fma_tflops || !h_ex2_tops || !d_sink) return TAOT_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    TAOT_CUDA_OK(cudaGetDevice(&dev));
    TAOT_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int blocks = sms * 8;                                  // 2048 threads per SM
    const int outer = 16;
    cudaEvent_t e0, e1;
    TAOT_CUDA_OK(cudaEventCreate(&e0));
    TAOT_CUDA_OK(cudaEventCreate(&e1));
    float best_fma = 0.0f, best_ex2 = 0.0f;
    for (int rep = 0; rep < 5; ++rep) {                          // first repetitions warm the clocks up
        float ms = 0.0f;
        cudaEventRecord(e0, st);
        fma_peak_kernel<<<blocks, kPeakThreads, 0, st>>>(static_cast<float*>(d_sink), outer, 0.999f, 1e-3f);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) {
            cudaEventDestroy(e0); cudaEventDestroy(e1);
            return TAOT_ERR_CUDA;
        }
        const double flops = 2.0 * (double)blocks * kPeakThreads * kChains * kInner * outer;
        const float t = (float)(flops / (ms * 1e-3) * 1e-12);
        if (t > best_fma) best_fma = t;
        cudaEventRecord(e0, st);
        ex2_peak_kernel<<<blocks, kPeakThreads, 0, st>>>(static_cast<float*>(d_sink), outer);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) {
            cudaEventDestroy(e0); cudaEventDestroy(e1);
            return TAOT_ERR_CUDA;
        }
        const double ops = (double)blocks * kPeakThreads * kChains * kInner * outer;
        const float x = (float)(ops / (ms * 1e-3) * 1e-12);
        if (x > best_ex2) best_ex2 = x;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *h_fma_tflops = best_fma;
    *h_ex2_tops = best_ex2;
    return TAOT_OK;
}

extern "C" int taot_measure_round_latencies(float* h_cycles, void* d_sink, void* stream)
{
    if (!h_cycles || !d_sink) return TAOT_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    round_latency_kernel<<<1, 256, 0, st>>>(static_cast<float*>(d_sink), 2048);
    TAOT_CUDA_OK(cudaGetLastError());
    float h[5];
    TAOT_CUDA_OK(cudaMemcpyAsync(h, d_sink, sizeof(h), cudaMemcpyDeviceToHost, st));
    TAOT_CUDA_OK(cudaStreamSynchronize(st));
    for (int i = 0; i < 4; ++i) h_cycles[i] = h[i];
    return TAOT_OK;
}
