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

// Status word of the resident-row kernel: waits that ran out leave their code here.
static __device__ unsigned int g_row_status;

namespace res {
unsigned int *row_status_word() {
  // one address per device; the symbol exists on every device that loads the library
  static unsigned int *cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cached[dev]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_row_status) != cudaSuccess) return nullptr;
    cached[dev] = static_cast<unsigned int *>(ptr);
  }
  return cached[dev];
}
}  // namespace res

cudaError_t read_and_clear_row_status(uint32_t *host_out) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(host_out, g_row_status, sizeof(uint32_t));
  if (e != cudaSuccess) return e;
  const unsigned int zero = 0;
  return cudaMemcpyToSymbol(g_row_status, &zero, sizeof(zero));
}

// Status word of the bounds-checking build.
static __device__ unsigned int g_bounds_status;

unsigned int *bounds_status_word() {
#ifdef DVP_DEBUG_BOUNDS
  static unsigned int *cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cached[dev]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_bounds_status) != cudaSuccess) return nullptr;
    cached[dev] = static_cast<unsigned int *>(ptr);
  }
  return cached[dev];
#else
  return nullptr;
#endif
}

cudaError_t read_and_clear_bounds_status(uint32_t *host_out) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(host_out, g_bounds_status, sizeof(uint32_t));
  if (e != cudaSuccess) return e;
  const unsigned int zero = 0;
  return cudaMemcpyToSymbol(g_bounds_status, &zero, sizeof(zero));
}

cudaError_t launch_row_kernels(const RowParams &p_in, int logits_dtype, int grad_dtype, uint32_t hint,
                               cudaStream_t s) {
  RowParams p = p_in;
  p.bounds_status = bounds_status_word();
  switch (logits_dtype) {
    case DVP_F32: return launch_row_kernels_f32(p, grad_dtype, hint, s);
    case DVP_BF16: return launch_row_kernels_bf16(p, grad_dtype, hint, s);
    default: return launch_row_kernels_f16(p, grad_dtype, hint, s);
  }
}

cudaError_t launch_backward_kernel(const BackwardParams &p_in, int logits_dtype, int grad_dtype,
                                   uint32_t hint, cudaStream_t s) {
  BackwardParams p = p_in;
  p.bounds_status = bounds_status_word();
  switch (logits_dtype) {
    case DVP_F32: return launch_backward_kernel_f32(p, grad_dtype, hint, s);
    case DVP_BF16: return launch_backward_kernel_bf16(p, grad_dtype, hint, s);
    default: return launch_backward_kernel_f16(p, grad_dtype, hint, s);
  }
}

}  // namespace dvp
