// Tensor-core path of the decomposed linear layer (placeholder until the tcgen05 kernel lands).
#include "linear.cuh"

namespace szo {

szo_status tc_plan_create(szo_linear* p, cudaStream_t) {
  p->tc = nullptr;
  return SZO_OK;
}

void tc_plan_destroy(szo_linear* p) { p->tc = nullptr; }

szo_status linear_fwd_tc(const szo_linear*, const void*, int64_t, const float*, void*, int, bool, cudaStream_t) {
  return fail(SZO_ERR_UNSUPPORTED, "tensor-core path not built");
}

}  // namespace szo
