// Host side of the C ABI: descriptor validation, plan object, dispatch to the kernel paths.
#include "common.cuh"

#include <math.h>
#include <stdio.h>
#include <string.h>
#include <new>

namespace darkattn {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e, const char *where)
{
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
}

void timer_mark(const darkattn_plan_s *plan, cudaStream_t st, const char *name)
{
    KernelTimer &t = plan->timer;
    if (!t.on || t.n >= KernelTimer::kMaxMarks) return;
    t.name[t.n] = name;
    cudaEventRecord(t.ev[t.n], st);
    ++t.n;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace darkattn

using namespace darkattn;

extern "C" {

darkattn_status_t darkattn_plan(const darkattn_desc_t *desc, darkattn_plan_t *out)
{
    if (!desc || !out) return DARKATTN_ERR_INVALID_ARG;
    *out = nullptr;
    darkattn_desc_t ds = *desc;
    if (ds.B < 1 || ds.H < 1 || ds.N < 1 || ds.d < 1 || ds.m < 1 || ds.r < 0 || ds.dv < 0 || ds.chunk < 0 || ds.H_kv < 0)
        return DARKATTN_ERR_INVALID_ARG;
    if (ds.H_kv == 0) ds.H_kv = ds.H;
    if (ds.H_kv > ds.H || ds.H % ds.H_kv) return DARKATTN_ERR_INVALID_ARG;
    if (ds.dtype != DARKATTN_F32 && ds.dtype != DARKATTN_BF16) return DARKATTN_ERR_INVALID_ARG;
    if (ds.path < DARKATTN_PATH_AUTO || ds.path > DARKATTN_PATH_TENSOR) return DARKATTN_ERR_INVALID_ARG;
    if (!(ds.scale >= 0.f) || !isfinite(ds.scale)) return DARKATTN_ERR_INVALID_ARG;
    if (ds.r == 0) ds.r = ds.d;
    if (ds.dv == 0) ds.dv = ds.d;
    if (ds.chunk == 0) ds.chunk = 128;
    if (ds.scale == 0.f) ds.scale = 1.0f / sqrtf((float)ds.d);
    if ((long long)ds.B * ds.H > 65535) return DARKATTN_ERR_UNSUPPORTED;

    darkattn_plan_s *p = new (std::nothrow) darkattn_plan_s();
    if (!p) return DARKATTN_ERR_INVALID_ARG;
    p->desc = ds;
    Dims &D = p->dims;
    D.B = ds.B; D.H = ds.H; D.N = ds.N; D.d = ds.d; D.r = ds.r; D.m = ds.m; D.dv = ds.dv;
    D.BH = ds.B * ds.H;
    D.Hkv = ds.H_kv; D.G = ds.H / ds.H_kv;
    D.causal = ds.causal ? 1 : 0;
    D.C = D.causal ? ds.chunk : ds.N;
    D.nc = D.causal ? (ds.N + D.C - 1) / D.C : 1;
    D.Npad = D.causal ? D.nc * D.C : ds.N;
    D.dva = ds.dv + 1;
    D.bf16 = ds.dtype == DARKATTN_BF16;
    D.w_per_head = ds.w_per_head ? 1 : 0;
    D.s = sqrtf(ds.scale);

    int path = ds.path;
    const bool tensor_ok = tensor_supported(p);
    if (path == DARKATTN_PATH_TENSOR && (!D.bf16 || !tensor_ok)) { delete p; return DARKATTN_ERR_UNSUPPORTED; }
    if (path == DARKATTN_PATH_AUTO) path = (D.bf16 && tensor_ok) ? DARKATTN_PATH_TENSOR : DARKATTN_PATH_SIMT;
    p->path = path;

    simt_make_layout(p);
    p->workspace_bytes = p->simt.total_bytes;
    p->saved_bytes = 0;
    {
        const int stage = (D.bf16 ? 5 : 0) + 4 + 6 + (D.causal ? 5 : 2);
        p->launches_fwd = stage + 1;
        p->launches_bwd = stage + (D.bf16 ? 1 : 0) + 1 + (D.causal ? 9 : 4) + 1 + 2 * 6 + 1;
    }
    if (path == DARKATTN_PATH_TENSOR) tensor_make_layout(p);
    *out = p;
    return DARKATTN_OK;
}

size_t darkattn_workspace_bytes(darkattn_plan_t plan) { return plan ? plan->workspace_bytes : 0; }
size_t darkattn_saved_bytes(darkattn_plan_t plan) { return plan ? plan->saved_bytes : 0; }
int32_t darkattn_plan_path(darkattn_plan_t plan) { return plan ? plan->path : -1; }
darkattn_status_t darkattn_forward(darkattn_plan_t plan, const void *Q, const void *K, const void *V,
                                   const void *M, const void *W, void *O, void *saved, void *workspace,
                                   void *cuda_stream)
{
    if (!plan || !Q || !K || !V || !M || !W || !O) return DARKATTN_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(M) || !aligned16(W) || !aligned16(O))
        return DARKATTN_ERR_INVALID_ARG;
    if (plan->workspace_bytes && !workspace) return DARKATTN_ERR_WORKSPACE;
    if (!aligned16(workspace) || !aligned16(saved)) return DARKATTN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DARKATTN_CUDA_TRY(cudaMemsetAsync(workspace, 0, 256, st), "forward: clear status word");
    darkattn_status_t rc;
    if (plan->path == DARKATTN_PATH_TENSOR) {
        rc = tensor_forward(plan, Q, K, V, M, W, O, saved, static_cast<char *>(workspace), st, saved != nullptr);
    } else {
        timer_mark(plan, st, "simt_forward (all kernels)");
        rc = simt_forward(plan, Q, K, V, M, W, O, static_cast<char *>(workspace), st, false);
    }
    timer_mark(plan, st, nullptr);
    return rc;
}

darkattn_status_t darkattn_backward(darkattn_plan_t plan, const void *Q, const void *K, const void *V,
                                    const void *M, const void *W, const void *O, const void *dO,
                                    const void *saved, void *dQ, void *dK, void *dV, float *dM,
                                    void *workspace, void *cuda_stream)
{
    if (!plan || !Q || !K || !V || !M || !W || !dO || !dQ || !dK || !dV || !dM) return DARKATTN_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(M) || !aligned16(W) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) || !aligned16(dM))
        return DARKATTN_ERR_INVALID_ARG;
    if (plan->workspace_bytes && !workspace) return DARKATTN_ERR_WORKSPACE;
    if (!aligned16(workspace) || !aligned16(saved) || !aligned16(O)) return DARKATTN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DARKATTN_CUDA_TRY(cudaMemsetAsync(workspace, 0, 256, st), "backward: clear status word");
    darkattn_status_t rc;
    if (plan->path == DARKATTN_PATH_TENSOR) {
        rc = tensor_backward(plan, Q, K, V, M, W, O, dO, saved, dQ, dK, dV, dM, static_cast<char *>(workspace), st);
    } else {
        timer_mark(plan, st, "simt_backward (all kernels)");
        rc = simt_backward(plan, Q, K, V, M, W, dO, dQ, dK, dV, dM, static_cast<char *>(workspace), st);
    }
    timer_mark(plan, st, nullptr);
    return rc;
}

darkattn_status_t darkattn_backward_dw(darkattn_plan_t plan, const void *M, float *dW, void *workspace, void *cuda_stream)
{
    if (!plan || !M || !dW || !workspace) return DARKATTN_ERR_INVALID_ARG;
    if (!aligned16(M) || !aligned16(dW) || !aligned16(workspace)) return DARKATTN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    darkattn_status_t rc = plan->path == DARKATTN_PATH_TENSOR
                               ? tensor_backward_dw(plan, M, dW, static_cast<char *>(workspace), st)
                               : simt_backward_dw(plan, dW, static_cast<char *>(workspace), st);
    timer_mark(plan, st, nullptr);
    return rc;
}

darkattn_status_t darkattn_last_device_status(darkattn_plan_t plan, const void *workspace, void *cuda_stream)
{
    if (!plan || !workspace) return DARKATTN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    DARKATTN_CUDA_TRY(cudaStreamSynchronize(st), "last_device_status: sync");
    DARKATTN_CUDA_TRY(cudaMemcpy(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost), "last_device_status: read");
    if (word == 0) return DARKATTN_OK;
    if (word == DARKATTN_ERR_NONFINITE || word == DARKATTN_ERR_CUDA) return (darkattn_status_t)word;
    return DARKATTN_ERR_TIMEOUT;
}

void darkattn_destroy(darkattn_plan_t plan)
{
    if (plan && plan->timer.created)
        for (int i = 0; i < KernelTimer::kMaxMarks; ++i) cudaEventDestroy(plan->timer.ev[i]);
    if (plan && plan->aux_stream) {
        cudaEventDestroy(plan->aux_fork);
        cudaEventDestroy(plan->aux_join);
        cudaStreamDestroy(plan->aux_stream);
    }
    delete plan;
}

const char *darkattn_status_string(darkattn_status_t s)
{
    switch (s) {
    case DARKATTN_OK: return "ok";
    case DARKATTN_ERR_INVALID_ARG: return "invalid argument";
    case DARKATTN_ERR_UNSUPPORTED: return "unsupported shape, dtype or path";
    case DARKATTN_ERR_WORKSPACE: return "workspace missing";
    case DARKATTN_ERR_CUDA: return "CUDA call failed";
    case DARKATTN_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case DARKATTN_ERR_NONFINITE: return "non-finite normaliser";
    }
    return "unknown status";
}

const char *darkattn_last_cuda_error(void) { return g_cuda_error; }

}  // extern "C"
