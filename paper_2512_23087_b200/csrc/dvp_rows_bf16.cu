// Row kernels instantiated for bf16 logits.
#include "dvp_rows_impl.cuh"

namespace dvp {

cudaError_t launch_row_kernels_bf16(const RowParams &p, int grad_dtype, uint32_t hint, cudaStream_t s) {
  return launch_rows_g<__nv_bfloat16>(p, grad_dtype, hint, s);
}

cudaError_t launch_backward_kernel_bf16(const BackwardParams &p, int grad_dtype, uint32_t hint,
                                          cudaStream_t s) {
  return launch_bwd_g<__nv_bfloat16>(p, grad_dtype, hint, s);
}

}  // namespace dvp
