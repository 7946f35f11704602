// Self-test of the bounded device-side wait every scan kernel uses: one thread waits on an mbarrier nobody ever
// arrives on. The wait gives up after its limit, records DARKATTN_ERR_TIMEOUT in a status word and returns; the
// kernel ends normally and the context stays usable.
#include "common.cuh"
#include "tc_common.cuh"

namespace darkattn {

using namespace tc;

namespace {

__device__ int g_selftest_status;

__global__ void wait_limit_kernel(int *status)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; fence_mbar_init(); }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool completed = wait_or_abort(&bar, 0, status, &abort_flag);
        if (completed) atomicExch(status, -1);      // cannot happen: nothing arrives on the barrier
    }
}

}  // namespace
}  // namespace darkattn

using namespace darkattn;

extern "C" darkattn_status_t darkattn_selftest_wait_limit(int32_t *device_status, double *seconds, void *cuda_stream)
{
    if (!device_status || !seconds) return DARKATTN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int *status = nullptr;
    DARKATTN_CUDA_TRY(cudaGetSymbolAddress((void **)&status, g_selftest_status), "selftest: symbol");
    DARKATTN_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int), st), "selftest: status");
    cudaEvent_t e0, e1;
    DARKATTN_CUDA_TRY(cudaEventCreate(&e0), "selftest: event");
    DARKATTN_CUDA_TRY(cudaEventCreate(&e1), "selftest: event");
    cudaEventRecord(e0, st);
    wait_limit_kernel<<<1, 32, 0, st>>>(status);
    cudaEventRecord(e1, st);
    int host = 0;
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(&host, status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) { set_cuda_error(e, "selftest: wait limit"); return DARKATTN_ERR_CUDA; }
    *device_status = host;
    *seconds = ms * 1e-3;
    return DARKATTN_OK;
}
