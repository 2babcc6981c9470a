// Row kernels instantiated for f16 logits.
#include "dvp_rows_impl.cuh"

namespace dvp {

cudaError_t launch_row_kernels_f16(const RowParams &p, int grad_dtype, uint32_t hint, cudaStream_t s) {
  return launch_rows_g<__half>(p, grad_dtype, hint, s);
}

cudaError_t launch_backward_kernel_f16(const BackwardParams &p, int grad_dtype, uint32_t hint,
                                          cudaStream_t s) {
  return launch_bwd_g<__half>(p, grad_dtype, hint, s);
}

}  // namespace dvp
