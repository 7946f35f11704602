// Microbenchmark of the tensor pipe as the scan kernels use it: cycles per 128 x N x 16 bf16 tcgen05.mma
// for the operand placements that occur (both operands in shared memory, K- or MN-major; A in tensor memory),
// optionally with the 16 epilogue warps reading tensor memory and writing shared memory beside the MMAs.
// One CTA per SM; one thread issues reps * 8 MMAs onto one accumulator, commits, and waits (bounded) for the commit.
#include "../csrc/common.cuh"
#include "../csrc/tc_common.cuh"
#include "darkattn_bench.h"

namespace darkattn {

using namespace tc;

namespace {

constexpr int kSmemBytes = 160 * 1024;     // A tile at 0 (32 KB), B tile at 32 KB (up to 64 KB), noise tile at 128 KB

__device__ long long g_cycles[1024];
__device__ int g_status;

// VARIANT: 0 SS K/K N=128, 1 SS K/MN, 2 SS MN/MN, 3 TS K, 4 TS MN, 5 SS K/K N=256, 6 SS K/K N=64, 7 SS MN/K N=16
template <int VARIANT>
__global__ void __launch_bounds__(kThreads, 1) mma_cycles_kernel(int reps, int busy, long long *out, int *status)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ uint64_t bar;
    __shared__ uint32_t slot;
    __shared__ int abort_flag;
    __shared__ volatile int done;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < kSmemBytes / 4; i += kThreads) reinterpret_cast<uint32_t *>(smem)[i] = 0x3C003C00u;   // small bf16 values
    if (tid == 0) { mbar_init(&bar, 1); abort_flag = 0; done = 0; fence_mbar_init(); }
    fence_async_smem();
    if (warp == kEpiWarps) { tmem_alloc(&slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = slot;
    if (tid == kEpiThreads) {
        const TileDesc tA(smem), tB(smem + 32768);
        constexpr int N = VARIANT == 5 ? 256 : VARIANT == 6 ? 64 : VARIANT == 7 ? 16 : 128;
        constexpr int a_mn = (VARIANT == 2 || VARIANT == 7) ? 1 : 0, b_mn = (VARIANT == 1 || VARIANT == 2 || VARIANT == 4) ? 1 : 0;
        const uint32_t idesc = make_idesc(128, N, a_mn, b_mn);
        const uint64_t b256 = make_sdesc(smem_u32(smem + 32768), 16, 1024);    // 256 rows: 64-element K blocks 32 KB apart
        const long long t0 = clock64();
        for (int rp = 0; rp < reps; ++rp) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (VARIANT == 0 || VARIANT == 6) mma_ss(tmem, kdesc(tA, k), kdesc(tB, k), idesc, 1);
                else if (VARIANT == 1) mma_ss(tmem, kdesc(tA, k), mndesc(tB, k), idesc, 1);
                else if (VARIANT == 2) mma_ss(tmem, mndesc(tA, k), mndesc(tB, k), idesc, 1);
                else if (VARIANT == 3) mma_ts(tmem, tmem + 256 + k * 8, kdesc(tB, k), idesc, 1);
                else if (VARIANT == 4) mma_ts(tmem, tmem + 256 + k * 8, mndesc(tB, k), idesc, 1);
                else if (VARIANT == 5) mma_ss(tmem, kdesc(tA, k), b256 + (uint64_t)(((k / 4) * 32768 + (k % 4) * 32) >> 4), idesc, 1);
                else mma_ss(tmem, mndesc(tA, k), kdesc(tB, k % 4), idesc, 1);
            }
        }
        mma_commit(&bar);
        const bool ok = wait_or_abort(&bar, 0, status, &abort_flag);
        out[blockIdx.x] = ok ? clock64() - t0 : -1;
        done = 1;
    } else if (warp < kEpiWarps && busy) {
        // what the epilogue warps do beside the MMAs: 32 columns out of tensor memory, 64 bytes into a swizzled tile
        const int lane = tid & 31, q4 = warp & 3, col0 = (warp >> 2) * 32, r = q4 * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        unsigned char *tile = smem + 128 * 1024;
        while (!done) {
            uint32_t v[32];
            tmem_ld32(lane_addr + 384 + col0, v);
            tmem_wait_ld();
#pragma unroll
            for (int q = 0; q < 4; ++q)
                *reinterpret_cast<uint4 *>(tile_chunk(tile, r, col0 / 8 + q)) = make_uint4(v[8 * q], v[8 * q + 1] + v[8 * q + 2], v[8 * q + 3] + v[8 * q + 4],
                                                                                         v[8 * q + 5] + v[8 * q + 6] + v[8 * q + 7]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kEpiWarps) tmem_dealloc(tmem, 512);
}

template <int V>
cudaError_t launch_variant(int blocks, int reps, int busy, long long *out, int *status, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(mma_cycles_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    mma_cycles_kernel<V><<<blocks, kThreads, kSmemBytes, st>>>(reps, busy, out, status);
    return cudaGetLastError();
}

}  // namespace
}  // namespace darkattn

using namespace darkattn;

extern "C" darkattn_status_t darkattn_measure_mma_cycles(int32_t variant, int32_t busy_epilogue, double *cycles_per_mma,
                                                         double *batch_overhead_cycles, void *cuda_stream)
{
    if (!cycles_per_mma || !batch_overhead_cycles || variant < 0 || variant > 7) return DARKATTN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int dev = 0, sms = 0;
    DARKATTN_CUDA_TRY(cudaGetDevice(&dev), "mma_cycles: device");
    DARKATTN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "mma_cycles: sm count");
    if (sms > 1024) sms = 1024;
    long long *out = nullptr;
    int *status = nullptr;
    DARKATTN_CUDA_TRY(cudaGetSymbolAddress((void **)&out, g_cycles), "mma_cycles: symbol");
    DARKATTN_CUDA_TRY(cudaGetSymbolAddress((void **)&status, g_status), "mma_cycles: symbol");
    DARKATTN_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int), st), "mma_cycles: status");
    double avg[2] = {0.0, 0.0};
    const int reps[2] = {4, 36};
    long long host[1024];
    for (int pass = 0; pass < 2; ++pass) {
        cudaError_t e = cudaSuccess;
        switch (variant) {
        case 0: e = launch_variant<0>(sms, reps[pass], busy_epilogue, out, status, st); break;
        case 1: e = launch_variant<1>(sms, reps[pass], busy_epilogue, out, status, st); break;
        case 2: e = launch_variant<2>(sms, reps[pass], busy_epilogue, out, status, st); break;
        case 3: e = launch_variant<3>(sms, reps[pass], busy_epilogue, out, status, st); break;
        case 4: e = launch_variant<4>(sms, reps[pass], busy_epilogue, out, status, st); break;
        case 5: e = launch_variant<5>(sms, reps[pass], busy_epilogue, out, status, st); break;
        case 6: e = launch_variant<6>(sms, reps[pass], busy_epilogue, out, status, st); break;
        default: e = launch_variant<7>(sms, reps[pass], busy_epilogue, out, status, st); break;
        }
        if (e == cudaSuccess) e = cudaMemcpyAsync(host, out, sizeof(long long) * sms, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) { set_cuda_error(e, "mma_cycles: launch"); return DARKATTN_ERR_CUDA; }
        for (int i = 0; i < sms; ++i) {
            if (host[i] < 0) return DARKATTN_ERR_TIMEOUT;
            avg[pass] += (double)host[i] / sms;
        }
    }
    // total(reps) = overhead + 8 reps c  at reps = 4 and 36
    *cycles_per_mma = (avg[1] - avg[0]) / (8.0 * (reps[1] - reps[0]));
    *batch_overhead_cycles = avg[0] - 8.0 * reps[0] * (*cycles_per_mma);
    return DARKATTN_OK;
}
