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

}  // namespace

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
