// Row kernels instantiated for f32 logits.
#include "dvp_rows_impl.cuh"

namespace dvp {

cudaError_t launch_row_kernels_f32(const RowParams &p, int grad_dtype, uint32_t hint, cudaStream_t s) {
  return launch_rows_g<float>(p, grad_dtype, hint, s);
}

cudaError_t launch_backward_kernel_f32(const BackwardParams &p, int grad_dtype, uint32_t hint,
                                          cudaStream_t s) {
  return launch_bwd_g<float>(p, grad_dtype, hint, s);
}

}  // namespace dvp
