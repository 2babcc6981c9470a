// C ABI of the DVP library: argument validation and kernel dispatch.
#include <cmath>

#include "dvp_common.cuh"

namespace {

bool dtype_ok(int d) { return d == DVP_F32 || d == DVP_BF16 || d == DVP_F16; }

bool hint_ok(uint32_t hint) {
  const uint32_t threads = hint & 0xffff, stage = (hint >> 16) & 0xff;
  if (threads != 0 && (threads % 32 != 0 || threads > 512)) return false;
  const uint32_t cluster = (hint >> 24) & 0xff;
  if (stage == 0x11 || stage == 0x1e) return cluster == 0;  // the resident-row kernel (0x1e: its self-test)
  return (stage == 0 || stage == 2 || stage == 3 || stage == 4) && (cluster == 0 || cluster == 1 || cluster == 2 || cluster == 4);
}

bool mode_ok(uint32_t mode, float mask_value) {
  if (mode & ~(uint32_t)(DVP_MODE_FINITE_MASK | DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE)) return false;
  return !(mode & DVP_MODE_FINITE_MASK) || std::isfinite(mask_value);
}

bool side_empty(const dvp_side_out &o) {
  return !o.max && !o.lse && !o.lse_safe && !o.logp && !o.logp_mp && !o.comp_mp && !o.count &&
         !o.mask && !o.log_cov;
}

double log_of_rho(double rho) { return rho > 0.0 ? std::log(rho) : -HUGE_VAL; }

}  // namespace

extern "C" {

int dvp_forward(const dvp_forward_args *a) {
  if (!a || a->struct_size != sizeof(dvp_forward_args)) return DVP_ERR_INVALID_ARG;
  if (!dtype_ok(a->logits_dtype)) return DVP_ERR_UNSUPPORTED;
  if (a->grad_train && !dtype_ok(a->grad_dtype)) return DVP_ERR_UNSUPPORTED;
  if (a->id_dtype != DVP_ID_I64 && a->id_dtype != DVP_ID_I32) return DVP_ERR_UNSUPPORTED;
  if (a->T < 0 || a->T > 0x7fffffffLL || a->V < 1) return DVP_ERR_INVALID_ARG;
  if (a->V > 0x7fffff00LL) return DVP_ERR_UNSUPPORTED;
  if (!(a->rho >= 0.0 && a->rho <= 1.0)) return DVP_ERR_INVALID_ARG;
  if (!hint_ok(a->launch_hint) || !mode_ok(a->mode, a->mask_value)) return DVP_ERR_INVALID_ARG;
  if (a->T == 0) return DVP_OK;
  if (!a->train_logits || a->ld_train < a->V) return DVP_ERR_INVALID_ARG;
  if (a->infer_logits && a->ld_infer < a->V) return DVP_ERR_INVALID_ARG;
  if (!a->infer_logits && (!side_empty(a->infer) || a->log_ratio)) return DVP_ERR_INVALID_ARG;
  if ((a->upstream != nullptr) != (a->grad_train != nullptr)) return DVP_ERR_INVALID_ARG;
  if (a->grad_train && (a->ld_grad < a->V || !a->ids)) return DVP_ERR_INVALID_ARG;
  if (a->weight_kind > DVP_WEIGHT_MASK) return DVP_ERR_INVALID_ARG;
  if (a->weight_kind != DVP_WEIGHT_NONE) {
    if (!a->infer_logits || !a->grad_train) return DVP_ERR_INVALID_ARG;
    if (!(a->weight_lo >= 0.f && a->weight_hi >= a->weight_lo)) return DVP_ERR_INVALID_ARG;
  } else if (a->weight_out) {
    return DVP_ERR_INVALID_ARG;
  }

  dvp::RowParams p{};
  p.train = a->train_logits;
  p.infer = a->infer_logits;
  p.ids = a->ids;
  p.upstream = a->upstream;
  p.grad = a->grad_train;
  p.T = a->T;
  p.V = a->V;
  p.ld_train = a->ld_train;
  p.ld_infer = a->ld_infer;
  p.ld_grad = a->ld_grad;
  p.log_rho = log_of_rho(a->rho);
  p.id_is_i32 = a->id_dtype == DVP_ID_I32;
  p.mode = (int)a->mode;
  p.mask_value = a->mask_value;
  p.out_t = a->train;
  p.out_i = a->infer;
  p.log_ratio = a->log_ratio;
  p.flags = a->flags;
  p.weight_kind = (int)a->weight_kind;
  p.weight_lo = a->weight_lo;
  p.weight_hi = a->weight_hi;
  p.weight_out = a->weight_out;
  const cudaError_t e = dvp::launch_row_kernels(p, a->logits_dtype, a->grad_dtype, a->launch_hint,
                                                static_cast<cudaStream_t>(a->stream));
  return e == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
}

int dvp_backward(const dvp_backward_args *a) {
  if (!a || a->struct_size != sizeof(dvp_backward_args)) return DVP_ERR_INVALID_ARG;
  if (!dtype_ok(a->logits_dtype) || !dtype_ok(a->grad_dtype)) return DVP_ERR_UNSUPPORTED;
  if (a->id_dtype != DVP_ID_I64 && a->id_dtype != DVP_ID_I32) return DVP_ERR_UNSUPPORTED;
  if (a->T < 0 || a->T > 0x7fffffffLL || a->V < 1) return DVP_ERR_INVALID_ARG;
  if (a->V > 0x7fffff00LL) return DVP_ERR_UNSUPPORTED;
  if (!(a->rho >= 0.0 && a->rho <= 1.0)) return DVP_ERR_INVALID_ARG;
  if (!hint_ok(a->launch_hint) || !mode_ok(a->mode, a->mask_value)) return DVP_ERR_INVALID_ARG;
  if (a->T == 0) return DVP_OK;
  if (!a->train_logits || !a->ids || !a->upstream || !a->max_t || !a->lse_safe_t || !a->flags ||
      !a->grad_train)
    return DVP_ERR_INVALID_ARG;
  if (a->ld_train < a->V || a->ld_grad < a->V) return DVP_ERR_INVALID_ARG;

  dvp::BackwardParams p{};
  p.train = a->train_logits;
  p.ids = a->ids;
  p.upstream = a->upstream;
  p.max_t = a->max_t;
  p.lse_safe_t = a->lse_safe_t;
  p.comp_mp_t = a->comp_mp_t;
  p.flags = a->flags;
  p.grad = a->grad_train;
  p.T = a->T;
  p.V = a->V;
  p.ld_train = a->ld_train;
  p.ld_grad = a->ld_grad;
  p.log_rho = log_of_rho(a->rho);
  p.id_is_i32 = a->id_dtype == DVP_ID_I32;
  p.mode = (int)a->mode;
  p.mask_value = a->mask_value;
  const cudaError_t e = dvp::launch_backward_kernel(p, a->logits_dtype, a->grad_dtype,
                                                    a->launch_hint,
                                                    static_cast<cudaStream_t>(a->stream));
  return e == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
}

int dvp_row_wait_status(uint32_t *status_out) {
  if (!status_out) return DVP_ERR_INVALID_ARG;
  return dvp::read_and_clear_row_status(status_out) == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
}

int dvp_debug_bounds_status(uint32_t *status_out) {
  if (!status_out) return DVP_ERR_INVALID_ARG;
#ifdef DVP_DEBUG_BOUNDS
  return dvp::read_and_clear_bounds_status(status_out) == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
#else
  *status_out = 0;
  return DVP_ERR_UNSUPPORTED;  // this library was built without the checks
#endif
}

const char *dvp_status_string(int status) {
  switch (status) {
    case DVP_OK: return "DVP_OK";
    case DVP_ERR_INVALID_ARG: return "DVP_ERR_INVALID_ARG";
    case DVP_ERR_UNSUPPORTED: return "DVP_ERR_UNSUPPORTED";
    case DVP_ERR_WORKSPACE: return "DVP_ERR_WORKSPACE";
    case DVP_ERR_CUDA: return "DVP_ERR_CUDA";
    default: return "DVP_ERR_UNKNOWN";
  }
}

int dvp_version(void) { return 200; }

}  // extern "C"
