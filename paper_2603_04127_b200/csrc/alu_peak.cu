// Register-only microbenchmarks for the two ALU resources behind the feature map's exponentials:
// MUFU ex2.approx.f32 and the FP32 FMA pipe. Their measured rates are the denominators of the
// exponent leg of the roofline.
#include "common.cuh"

namespace darkattn {
namespace {

constexpr int kChains = 8;
constexpr int kInner = 2048;

__global__ void __launch_bounds__(512) ex2_peak_kernel(float *sink, float seed)
{
    float x[kChains];
#pragma unroll
    for (int i = 0; i < kChains; ++i) x[i] = seed * (float)(threadIdx.x + i) * 1e-3f - 3.f;
    for (int it = 0; it < kInner; ++it) {
#pragma unroll
        for (int i = 0; i < kChains; ++i) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i]));
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kChains; ++i) acc += x[i];
    if (acc == 123.456f) sink[0] = acc;   // keeps the chains alive; practically never true
}

__global__ void __launch_bounds__(512) fma_peak_kernel(float *sink, float seed)
{
    float x[kChains];
#pragma unroll
    for (int i = 0; i < kChains; ++i) x[i] = seed * (float)(threadIdx.x + i);
    const float a = 0.999f + seed * 1e-9f, b = 1e-3f;
    for (int it = 0; it < kInner; ++it) {
#pragma unroll
        for (int i = 0; i < kChains; ++i) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(x[i]) : "f"(a), "f"(b));
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kChains; ++i) acc += x[i];
    if (acc == 123.456f) sink[0] = acc;
}

__device__ float g_sink[4];

}  // namespace
}  // namespace darkattn

using namespace darkattn;

extern "C" darkattn_status_t darkattn_measure_alu_peak(int32_t which, int32_t iters, double *ops_per_second,
                                                       void *cuda_stream)
{
    if (!ops_per_second || iters < 1 || which < 0 || which > 1) return DARKATTN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int dev = 0, sms = 0;
    DARKATTN_CUDA_TRY(cudaGetDevice(&dev), "alu_peak: device");
    DARKATTN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "alu_peak: sm count");
    float *sink = nullptr;
    DARKATTN_CUDA_TRY(cudaGetSymbolAddress((void **)&sink, g_sink), "alu_peak: symbol");
    const int blocks = sms * 4, threads = 512;
    cudaEvent_t e0, e1;
    DARKATTN_CUDA_TRY(cudaEventCreate(&e0), "alu_peak: event");
    DARKATTN_CUDA_TRY(cudaEventCreate(&e1), "alu_peak: event");
    auto launch = [&]() {
        if (which == 0) ex2_peak_kernel<<<blocks, threads, 0, st>>>(sink, 1.0f);
        else fma_peak_kernel<<<blocks, threads, 0, st>>>(sink, 1.0f);
    };
    for (int i = 0; i < 2; ++i) launch();
    cudaEventRecord(e0, st);
    for (int i = 0; i < iters; ++i) launch();
    cudaEventRecord(e1, st);
    cudaError_t e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) { set_cuda_error(e, "alu_peak: timing"); return DARKATTN_ERR_CUDA; }
    const double ops = (double)blocks * threads * (double)kChains * kInner * iters;
    *ops_per_second = ops / (ms * 1e-3);
    return DARKATTN_OK;
}
