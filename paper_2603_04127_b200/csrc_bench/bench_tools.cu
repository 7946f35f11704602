// Instruments of the benchmark and of the profiling runs, kept out of the product library: per-kernel device times
// (the product's launch code records events at every kernel while a plan's timer is on; these calls switch it on and
// harvest it) and the number of launches of a call. Built into libdarkattn_bench.so, which links against libdarkattn.so.
#include "../csrc/common.cuh"
#include "darkattn_bench.h"

#include <stdio.h>
#include <string.h>

using namespace darkattn;

extern "C" {

int32_t darkattn_plan_launches(darkattn_plan_t plan, int32_t which)
{
    if (!plan) return -1;
    if (!which) return plan->launches_fwd;
    // with per-kernel timing on, the tensor-core backward keeps everything on one stream and dM is one kernel, not two
    return plan->launches_bwd - ((plan->path == DARKATTN_PATH_TENSOR && plan->timer.on) ? 1 : 0);
}

darkattn_status_t darkattn_kernel_timing(darkattn_plan_t plan, int32_t enable)
{
    if (!plan) return DARKATTN_ERR_INVALID_ARG;
    KernelTimer &t = plan->timer;
    if (enable && !t.created) {
        for (int i = 0; i < KernelTimer::kMaxMarks; ++i)
            DARKATTN_CUDA_TRY(cudaEventCreate(&t.ev[i]), "kernel_timing: cudaEventCreate");
        t.created = true;
    }
    t.on = enable != 0;
    t.n = 0;
    if (enable) t.nk = 0;
    return DARKATTN_OK;
}

darkattn_status_t darkattn_kernel_times(darkattn_plan_t plan, int32_t max_entries, char *names, float *total_ms,
                                        int32_t *launches, int32_t *count)
{
    if (!plan || !names || !total_ms || !launches || !count || max_entries < 0) return DARKATTN_ERR_INVALID_ARG;
    KernelTimer &t = plan->timer;
    if (t.n > 0) {
        DARKATTN_CUDA_TRY(cudaEventSynchronize(t.ev[t.n - 1]), "kernel_times: cudaEventSynchronize");
        for (int i = 0; i + 1 < t.n; ++i) {
            if (!t.name[i]) continue;
            float ms = 0.f;
            DARKATTN_CUDA_TRY(cudaEventElapsedTime(&ms, t.ev[i], t.ev[i + 1]), "kernel_times: cudaEventElapsedTime");
            int k = 0;
            while (k < t.nk && strcmp(t.kname[k], t.name[i]) != 0) ++k;
            if (k == t.nk) {
                if (t.nk == KernelTimer::kMaxKernels) continue;
                t.kname[k] = t.name[i]; t.kms[k] = 0.0; t.kcount[k] = 0; ++t.nk;
            }
            t.kms[k] += ms;
            ++t.kcount[k];
        }
        t.n = 0;
    }
    const int n = t.nk < max_entries ? t.nk : max_entries;
    for (int k = 0; k < n; ++k) {
        snprintf(names + 64 * k, 64, "%s", t.kname[k]);
        total_ms[k] = (float)t.kms[k];
        launches[k] = t.kcount[k];
    }
    *count = n;
    return DARKATTN_OK;
}

}  // extern "C"
