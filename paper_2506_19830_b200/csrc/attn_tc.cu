// Tensor-core nested-prefix attention (placeholder until the tcgen05 kernel lands).
#include "lr_common.cuh"

namespace lr {

int init_attn_tc_kernel() { return LR_OK; }

int tc_build_host_plan(const lr_ctx *, const lr_batch *, const int32_t *, TcHostPlan &out, Image &) {
  out = TcHostPlan();
  return LR_OK;
}

void tc_bind_device_plan(const TcHostPlan &h, unsigned char *, unsigned char *, lr_plan *p) {
  p->tc_ok = h.ok;
  memset(&p->tc, 0, sizeof(p->tc));
}

int launch_attn_tc(lr_plan *, const void *, const void *, const void *, void *, float *, float, cudaStream_t) {
  set_error("tensor-core attention path not built");
  return LR_EUNSUPPORTED;
}

}  // namespace lr
