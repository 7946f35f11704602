// Tensor-core path of libdarkattn (tcgen05 MMA with TMEM accumulators, operands staged by TMA).
#include "common.cuh"

namespace darkattn {

bool tensor_supported(const darkattn_plan_s *) { return false; }
void tensor_make_layout(darkattn_plan_s *) {}

darkattn_status_t tensor_forward(const darkattn_plan_s *, const void *, const void *, const void *, const void *,
                                 const void *, void *, char *, cudaStream_t)
{
    return DARKATTN_ERR_UNSUPPORTED;
}

darkattn_status_t tensor_backward(const darkattn_plan_s *, const void *, const void *, const void *, const void *,
                                  const void *, const void *, void *, void *, void *, float *, char *, cudaStream_t)
{
    return DARKATTN_ERR_UNSUPPORTED;
}

}  // namespace darkattn
