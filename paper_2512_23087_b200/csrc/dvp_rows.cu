// Dispatch of the row kernels on the logits type; the kernels themselves are in
// dvp_rows_impl.cuh and are compiled once per type in dvp_rows_{f32,bf16,f16}.cu.
#include "dvp_common.cuh"

namespace dvp {

cudaError_t launch_row_kernels_f32(const RowParams &, int, uint32_t, cudaStream_t);
cudaError_t launch_row_kernels_bf16(const RowParams &, int, uint32_t, cudaStream_t);
cudaError_t launch_row_kernels_f16(const RowParams &, int, uint32_t, cudaStream_t);
cudaError_t launch_backward_kernel_f32(const BackwardParams &, int, uint32_t, cudaStream_t);
cudaError_t launch_backward_kernel_bf16(const BackwardParams &, int, uint32_t, cudaStream_t);
cudaError_t launch_backward_kernel_f16(const BackwardParams &, int, uint32_t, cudaStream_t);

cudaError_t launch_row_kernels(const RowParams &p, int logits_dtype, int grad_dtype, uint32_t hint,
                               cudaStream_t s) {
  switch (logits_dtype) {
    case DVP_F32: return launch_row_kernels_f32(p, grad_dtype, hint, s);
    case DVP_BF16: return launch_row_kernels_bf16(p, grad_dtype, hint, s);
    default: return launch_row_kernels_f16(p, grad_dtype, hint, s);
  }
}

cudaError_t launch_backward_kernel(const BackwardParams &p, int logits_dtype, int grad_dtype,
                                   uint32_t hint, cudaStream_t s) {
  switch (logits_dtype) {
    case DVP_F32: return launch_backward_kernel_f32(p, grad_dtype, hint, s);
    case DVP_BF16: return launch_backward_kernel_bf16(p, grad_dtype, hint, s);
    default: return launch_backward_kernel_f16(p, grad_dtype, hint, s);
  }
}

}  // namespace dvp
