// Fused LM-head entry point (placeholder until the tensor-core path lands).
#include "dvp_common.cuh"

extern "C" {

int dvp_fused_lmhead_forward_backward(const dvp_fused_args *a) {
  if (!a || a->struct_size != sizeof(dvp_fused_args)) return DVP_ERR_INVALID_ARG;
  return DVP_ERR_UNSUPPORTED;
}

size_t dvp_workspace_bytes(int entry_point, const void *args) {
  (void)entry_point;
  (void)args;
  return 0;
}

}  // extern "C"
