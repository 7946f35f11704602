// darkattn_forward_static: the forward pass for callers that cannot provide (or allocate) a workspace.
//
// Its scratch is a fixed array in the library's own device image. The array is shared by every call
// on a device and keeps whatever the previous call left in it.
#include "common.cuh"

#include <mutex>

namespace darkattn {
namespace {

// Scratch of the static entry point: DARKATTN_STATIC_SCRATCH_BYTES of device memory per GPU context
// that loads the library, resident until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[DARKATTN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
char *g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` names a host-side shadow of the symbol, not device memory, so the
// address kernels may use has to be asked for, with the target device current.
darkattn_status_t scratch_for_current_device(char **out)
{
    int dev = -1;
    DARKATTN_CUDA_TRY(cudaGetDevice(&dev), "forward_static: cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return DARKATTN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        DARKATTN_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch), "forward_static: cudaGetSymbolAddress");
        if (!p) return DARKATTN_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<char *>(p);
    }
    *out = g_scratch_addr[dev];
    return DARKATTN_OK;
}

}  // namespace
}  // namespace darkattn

using namespace darkattn;

extern "C" size_t darkattn_static_scratch_needed(darkattn_plan_t plan)
{
    return plan ? plan->simt.fwd_bytes : 0;
}

extern "C" darkattn_status_t darkattn_forward_static(darkattn_plan_t plan, const void *Q, const void *K,
                                                     const void *V, const void *M, const void *W, void *O,
                                                     void *cuda_stream)
{
    if (!plan || !Q || !K || !V || !M || !W || !O) return DARKATTN_ERR_INVALID_ARG;
    const void *ptrs[6] = {Q, K, V, M, W, O};
    for (const void *p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) & 15u) return DARKATTN_ERR_INVALID_ARG;
    // size check first: it needs no GPU, so a refusal never touches the device
    if (plan->simt.fwd_bytes > (size_t)DARKATTN_STATIC_SCRATCH_BYTES) return DARKATTN_ERR_WORKSPACE;
    char *scratch = nullptr;
    darkattn_status_t s = scratch_for_current_device(&scratch);
    if (s != DARKATTN_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array still holds the previous call's data: the status word must start at zero; every other
    // region is written by this call before it is read (the per-feature maxima are re-initialised by
    // the forward stages themselves)
    DARKATTN_CUDA_TRY(cudaMemsetAsync(scratch, 0, 256, st), "forward_static: clear status word");
    return simt_forward(plan, Q, K, V, M, W, O, scratch, st, false);
}
