// Fused LM-head entry point: z = hidden x W_vocab^T on the tensor cores, the
// row computation of dvp_forward on panels of those logits, and the chain rule
// through the head (d_hidden = G W, d_w = G^T hidden) as two more contractions.
//
// The [T, V] training logits are never stored: a panel of `panel_rows` tokens
// lives in the workspace as fp32 logits, is read once by the panel's row pass
// (dvp_panel.cuh), which leaves the per-token results and the gradient panel up to
// one factor per row, and that panel is consumed by the two gradient contractions
// before the next panel overwrites it.
//
// The panel is held in float16 (11-bit significand; bfloat16's 8 bits would miss
// the 1e-3 gradient tolerance by themselves): P = 2^14 e^{z - m} on the safe set.
// The factor per row, -g / (2^14 s_S), multiplies the rows of d_hidden in the
// contraction's epilogue and, times a power of two chosen from max |upstream|, the
// hidden rows as they are converted to float16 for the d_w contraction; the inverse
// power of two is applied in that contraction's epilogue.  tcgen05 kind::f16 needs
// both operands of one type, so W^T is converted to a float16 copy once per call
// (exact for bfloat16 values in float16's normal range).
#include <cmath>
#include <mutex>

#include "dvp_common.cuh"
#include "dvp_gemm.cuh"
#include "dvp_panel.cuh"

namespace dvp {

// out[c, r] = convert(in[r, c]) for a row-major [R, C] input of a 16-bit type.
// 64 x 64 tiles through shared memory; 16-byte accesses on both sides when the
// strides and bases allow it (ld_in, ld_out multiples of 8, 16-byte aligned bases).
template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256)
transpose_convert_kernel(const TIn *in, long long ld_in, TOut *out, long long ld_out, int R, int C,
                         int vec_ok, const float *row_scale) {
  __shared__ TOut tile[64][66];
  const int c0 = blockIdx.x * 64, r0 = blockIdx.y * 64;
  const int tid = threadIdx.x;
  // load: 64 rows x 8 vectors of 8 elements, two vectors per thread
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int v = tid + i * 256, r = r0 + (v >> 3), c = c0 + (v & 7) * 8;
    TOut e[8];
    const float rs = (row_scale && r < R) ? row_scale[r] : 1.f;  // input row r times rs
    if (vec_ok && r < R && c + 8 <= C) {
      const uint4 raw = *reinterpret_cast<const uint4 *>(in + (long long)r * ld_in + c);
      const TIn *x = reinterpret_cast<const TIn *>(&raw);
#pragma unroll
      for (int j = 0; j < 8; ++j) e[j] = Storage<TOut>::narrow(Storage<TIn>::widen(x[j]) * rs);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j)
        e[j] = (r < R && c + j < C)
                   ? Storage<TOut>::narrow(Storage<TIn>::widen(in[(long long)r * ld_in + c + j]) * rs)
                   : Storage<TOut>::narrow(0.f);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) tile[v >> 3][(v & 7) * 8 + j] = e[j];
  }
  __syncthreads();
  // store: 64 output rows (input columns) x 8 vectors of 8 input rows
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int v = tid + i * 256, c = c0 + (v >> 3), r = r0 + (v & 7) * 8;
    if (c >= C) continue;
    __align__(16) TOut e[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) e[j] = tile[(v & 7) * 8 + j][v >> 3];
    TOut *dst = out + (long long)c * ld_out + r;
    if (vec_ok && r + 8 <= R) {
      *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(e);
    } else {
      for (int j = 0; j < 8 && r + j < R; ++j) dst[j] = e[j];
    }
  }
}

template <typename TIn, typename TOut>
static void launch_transpose(const TIn *in, long long ld_in, TOut *out, long long ld_out, int R, int C,
                             cudaStream_t s, const float *row_scale = nullptr) {
  const int vec_ok = ld_in % 8 == 0 && ld_out % 8 == 0 && (uintptr_t)in % 16 == 0 && (uintptr_t)out % 16 == 0;
  transpose_convert_kernel<TIn, TOut>
      <<<dim3((C + 63) / 64, (R + 63) / 64), 256, 0, s>>>(in, ld_in, out, ld_out, R, C, vec_ok, row_scale);
}

struct FusedScalars {
  int status;       // non-zero when a tensor-core kernel gave up waiting
  float scale;      // power of two applied to the gradient panel
  float inv_scale;  // its inverse
};

// scale = 2^(14 - x) with max|g| < 2^x, so that |scale * G| < 2^14.
// `factor` bounds what the kernel multiplies into the upstream gradients (an importance weight).
__global__ void grad_scale_kernel(const float *upstream, long long T, float factor, FusedScalars *out) {
  __shared__ float red[32];
  float m = 0.f;
  for (long long t = threadIdx.x; t < T; t += blockDim.x) {
    const float v = fabsf(upstream[t]);
    if (v < __int_as_float(0x7f800000)) m = fmaxf(m, v);
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) m = fmaxf(m, red[w]);
    m *= factor;
    int x = 0;
    if (m > 0.f) frexpf(m, &x);
    int e = 14 - x;
    e = e > 60 ? 60 : (e < -60 ? -60 : e);
    out->status = 0;
    out->scale = ldexpf(1.f, e);
    out->inv_scale = ldexpf(1.f, -e);
  }
}

// Merge the two sides: flags and the per-token log-ratio.
__global__ void combine_sides_kernel(long long T, const float *lp_t, const float *lp_i,
                                     const uint8_t *flags_i, uint8_t *flags, float *log_ratio) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  const uint8_t ft = flags[t];
  const bool in_t = ft & DVP_FLAG_IN_TRAIN, in_i = flags_i[t] & DVP_FLAG_IN_TRAIN;
  flags[t] = (uint8_t)(ft | (in_i ? DVP_FLAG_IN_INFER : 0));
  if (log_ratio)
    log_ratio[t] = (ft & (DVP_FLAG_NO_ID | DVP_FLAG_BAD_ID)) ? __int_as_float(0x7fc00000)
                                                             : log_ratio_of(in_t, in_i, lp_t[t], lp_i[t]);
}

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct FusedLayout {
  long long Vp, Tp, panel;
  size_t off_scalars, off_lpt, off_lpi, off_fli, off_flt, off_wt, off_hs, off_z, off_g, off_rmax, off_rowscale,
      off_hidscale, off_acoef, off_sort, total;
  long long max_pieces;
};

bool fused_layout(const dvp_fused_args *a, FusedLayout *L) {
  if (a->T < 0 || a->H < 1 || a->V < 1) return false;
  long long panel = a->panel_rows;
  if (panel == 0) {
    panel = (a->T + 127) / 128 * 128;
    if (panel > 4096) panel = 4096;
    if (panel < 128) panel = 128;
  }
  if (panel % 128 != 0 || panel < 128) return false;
  L->panel = panel;
  L->Vp = (a->V + 15) / 16 * 16;
  L->Tp = (a->T + 7) / 8 * 8;
  if (L->Tp == 0) L->Tp = 8;
  size_t o = 0;
  auto take = [&](size_t bytes) {
    const size_t at = o;
    o = align_up(o + bytes, 256);
    return at;
  };
  L->off_scalars = take(sizeof(FusedScalars));
  L->off_lpt = take((size_t)a->T * 4);
  L->off_lpi = take((size_t)a->T * 4);
  L->off_fli = take((size_t)a->T);
  L->off_flt = take((size_t)a->T);
  L->off_wt = take((size_t)a->H * L->Vp * 2);
  L->off_hs = take((size_t)a->H * panel * 2);  // the panel's hidden rows, scaled, transposed, float16
  L->off_z = take((size_t)panel * L->Vp * 4);
  L->off_g = take((size_t)panel * L->Vp * 2);
  L->max_pieces = (a->V + gemm::kBN - 1) / gemm::kBN;  // one per tile column of the logits contraction
  L->off_rmax = take((size_t)panel * L->max_pieces * 4);
  L->off_rowscale = take((size_t)panel * 4);
  L->off_hidscale = take((size_t)panel * 4);
  L->off_acoef = take((size_t)panel * 4);
  L->off_sort = take((size_t)panel::kSortChunk * 8);
  L->total = o;
  return true;
}

dvp_side_out offset_side(const dvp_side_out &o, long long r0, long long words) {
  dvp_side_out r = o;
  if (r.max) r.max += r0;
  if (r.lse) r.lse += r0;
  if (r.lse_safe) r.lse_safe += r0;
  if (r.logp) r.logp += r0;
  if (r.logp_mp) r.logp_mp += r0;
  if (r.comp_mp) r.comp_mp += r0;
  if (r.count) r.count += r0;
  if (r.log_cov) r.log_cov += r0;
  if (r.mask) r.mask += r0 * words;
  return r;
}

}  // namespace
}  // namespace dvp

extern "C" {

size_t dvp_workspace_bytes(int entry_point, const void *args) {
  if (entry_point != DVP_ENTRY_FUSED_LMHEAD || !args) return 0;
  const dvp_fused_args *a = static_cast<const dvp_fused_args *>(args);
  if (a->struct_size != sizeof(dvp_fused_args)) return 0;
  dvp::FusedLayout L;
  return dvp::fused_layout(a, &L) ? L.total : 0;
}

int dvp_gemm_tn(const void *a, int64_t lda, const void *b, int64_t ldb, float *c, int64_t ldc, int64_t m,
                int64_t n, int64_t k, int32_t dtype, float alpha, int32_t accumulate, int32_t *status,
                void *stream) {
  if (!a || !b || !c || !status || m < 0 || n < 0 || k < 0) return DVP_ERR_INVALID_ARG;
  if (m > 0x7fffffffLL || n > 0x7fffffffLL || k > 0x7fffffffLL) return DVP_ERR_UNSUPPORTED;
  if (dtype != DVP_BF16 && dtype != DVP_F16) return DVP_ERR_UNSUPPORTED;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return DVP_ERR_CUDA;
  const cudaError_t e =
      dvp::gemm::launch_gemm_tn(a, lda, b, ldb, c, ldc, (int)m, (int)n, (int)k, dtype == DVP_BF16, alpha,
                                nullptr, (accumulate & 1) != 0, status, sms,
                                static_cast<cudaStream_t>(stream), (accumulate & 2) != 0, (accumulate & 4) != 0,
                                (accumulate & 8) ? 2 : 1);
  if (e == cudaErrorInvalidValue) return DVP_ERR_UNSUPPORTED;
  return e == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
}

int dvp_fused_lmhead_forward_backward(const dvp_fused_args *a) {
  using namespace dvp;
  if (!a || a->struct_size != sizeof(dvp_fused_args)) return DVP_ERR_INVALID_ARG;
  if (a->id_dtype != DVP_ID_I64 && a->id_dtype != DVP_ID_I32) return DVP_ERR_UNSUPPORTED;
  if (a->T < 0 || a->T > 0x7fffffffLL || a->H < 1 || a->V < 1) return DVP_ERR_INVALID_ARG;
  if (a->V > 0x7fffff00LL || a->H > 0x7fffff00LL) return DVP_ERR_UNSUPPORTED;
  if (!(a->rho >= 0.0 && a->rho <= 1.0)) return DVP_ERR_INVALID_ARG;
  FusedLayout L;
  if (!fused_layout(a, &L)) return DVP_ERR_INVALID_ARG;
  if (a->T == 0) return DVP_OK;
  if (!a->hidden || !a->w_vocab || !a->ids || !a->upstream || !a->d_hidden || !a->d_w)
    return DVP_ERR_INVALID_ARG;
  if (a->ld_hidden < a->H || a->ld_w < a->H || a->ld_dh < a->H || a->ld_dw < a->H)
    return DVP_ERR_INVALID_ARG;
  if (a->infer_logits && a->ld_infer < a->V) return DVP_ERR_INVALID_ARG;
  if (!a->infer_logits && a->log_ratio) return DVP_ERR_INVALID_ARG;
  if (a->weight_kind != DVP_WEIGHT_NONE) {
    if (a->weight_kind != DVP_WEIGHT_TRUNCATE && a->weight_kind != DVP_WEIGHT_MASK) return DVP_ERR_INVALID_ARG;
    if (!a->infer_logits) return DVP_ERR_INVALID_ARG;
    if (!(a->weight_lo >= 0.f && a->weight_hi >= a->weight_lo) || !std::isfinite(a->weight_hi))
      return DVP_ERR_INVALID_ARG;
  } else if (a->weight_out) {
    return DVP_ERR_INVALID_ARG;
  }
  if (a->ld_hidden % 8 || a->ld_w % 8 || a->ld_dh % 8 || a->ld_dw % 8 ||
      (uintptr_t)a->hidden % 16 || (uintptr_t)a->w_vocab % 16 || (uintptr_t)a->d_hidden % 32 ||
      (uintptr_t)a->d_w % 32)
    return DVP_ERR_UNSUPPORTED;
  if (!a->workspace || (uintptr_t)a->workspace % 256 || a->workspace_bytes < L.total)
    return DVP_ERR_WORKSPACE;

  cudaStream_t s = static_cast<cudaStream_t>(a->stream);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return DVP_ERR_CUDA;

  char *ws = static_cast<char *>(a->workspace);
  FusedScalars *sc = reinterpret_cast<FusedScalars *>(ws + L.off_scalars);
  float *lpt = a->train.logp_mp ? a->train.logp_mp : reinterpret_cast<float *>(ws + L.off_lpt);
  float *lpi = a->infer.logp_mp ? a->infer.logp_mp : reinterpret_cast<float *>(ws + L.off_lpi);
  uint8_t *fli = reinterpret_cast<uint8_t *>(ws + L.off_fli);
  uint8_t *flt = a->flags ? a->flags : reinterpret_cast<uint8_t *>(ws + L.off_flt);
  __half *wt16 = reinterpret_cast<__half *>(ws + L.off_wt);   // [H, Vp]: W^T
  __half *hs16 = reinterpret_cast<__half *>(ws + L.off_hs);   // [H, panel]: the panel's hidden rows, scaled, transposed
  float *z = reinterpret_cast<float *>(ws + L.off_z);         // [panel, Vp] logits
  __half *p16 = reinterpret_cast<__half *>(ws + L.off_g);     // [panel, Vp] P = 2^14 e^{z - m} on the safe set
  float *rmax = reinterpret_cast<float *>(ws + L.off_rmax);   // [panel, max_pieces] row maxima of z in pieces
  float *row_scale = reinterpret_cast<float *>(ws + L.off_rowscale);  // [panel] factor of each row of P
  float *hid_scale = reinterpret_cast<float *>(ws + L.off_hidscale);  // [panel] the same times a power of two
  float *a_coef = reinterpret_cast<float *>(ws + L.off_acoef);        // [panel] coefficient of the 1[k = a] term
  unsigned long long *sorted = reinterpret_cast<unsigned long long *>(ws + L.off_sort);
  const __nv_bfloat16 *hidden = static_cast<const __nv_bfloat16 *>(a->hidden);
  const __nv_bfloat16 *w = static_cast<const __nv_bfloat16 *>(a->w_vocab);
  const int T = (int)a->T, H = (int)a->H, V = (int)a->V;
  const long long id_bytes = a->id_dtype == DVP_ID_I32 ? 4 : 8;
  const long long mask_words = (a->V + 31) / 32;

  const bool weighted = a->weight_kind != DVP_WEIGHT_NONE;
  grad_scale_kernel<<<1, 1024, 0, s>>>(a->upstream, a->T, weighted ? fmaxf(1.f, a->weight_hi) : 1.f, sc);
  launch_transpose<__nv_bfloat16, __half>(w, a->ld_w, wt16, L.Vp, V, H, s);
  if (cudaGetLastError() != cudaSuccess) return DVP_ERR_CUDA;

  const double log_rho = a->rho > 0.0 ? std::log(a->rho) : -HUGE_VAL;
  // the inference rows: an ordinary forward-only row pass over the stored logits
  auto infer_rows = [&]() -> cudaError_t {
    RowParams p{};
    p.train = a->infer_logits;
    p.ids = a->ids;
    p.T = a->T;
    p.V = a->V;
    p.ld_train = a->ld_infer;
    p.log_rho = log_rho;
    p.id_is_i32 = a->id_dtype == DVP_ID_I32;
    p.out_t = a->infer;
    p.out_t.logp_mp = lpi;
    p.flags = fli;
    return launch_row_kernels(p, DVP_BF16, DVP_BF16, 0, s);
  };
  // with an importance weight the training rows need the inference side first
  if (weighted && infer_rows() != cudaSuccess) return DVP_ERR_CUDA;
  int panel_index = 0;
  for (long long r0 = 0; r0 < a->T; r0 += L.panel, ++panel_index) {
    const int rows = (int)((a->T - r0 < L.panel) ? a->T - r0 : L.panel);
    // logits of the panel: z = hidden[r0 : r0 + rows] x W^T (bf16 operands, fp32 accumulate)
    // its epilogue also leaves each row's maximum, one piece per tile column: the panel's row pass
    // then knows the threshold before it reads the panel
    cudaError_t e = gemm::launch_gemm_tn(hidden + r0 * a->ld_hidden, a->ld_hidden, w, a->ld_w, z, L.Vp,
                                         rows, V, H, true, 1.f, nullptr, false, &sc->status, sms, s, false,
                                         false, 1, rmax, L.max_pieces);
    if (e != cudaSuccess) return e == cudaErrorInvalidValue ? DVP_ERR_UNSUPPORTED : DVP_ERR_CUDA;
    // rows of the panel, one sweep: statistics, and the gradient panel up to a factor per row
    panel::PanelParams pp{};
    RowParams &p = pp.row;
    p.train = z;
    p.ids = static_cast<const char *>(a->ids) + r0 * id_bytes;
    p.upstream = a->upstream + r0;
    p.T = rows;
    p.V = a->V;
    p.ld_train = L.Vp;
    p.log_rho = log_rho;
    p.id_is_i32 = a->id_dtype == DVP_ID_I32;
    p.out_t = offset_side(a->train, r0, mask_words);
    p.out_t.logp_mp = lpt + r0;
    p.flags = flt + r0;
    p.bounds_status = bounds_status_word();
    if (weighted) {
      p.weight_kind = (int)a->weight_kind;
      p.weight_lo = a->weight_lo;
      p.weight_hi = a->weight_hi;
      p.weight_out = a->weight_out ? a->weight_out + r0 : nullptr;
      p.given_logp_mp_i = lpi + r0;
      p.given_flags_i = fli + r0;
    }
    pp.row_max = rmax;
    pp.row_max_ld = L.max_pieces;
    pp.row_max_n = (int)L.max_pieces;
    pp.P = p16;
    pp.ld_p = L.Vp;
    pp.row_scale = row_scale;
    pp.hid_scale = hid_scale;
    pp.a_coef = a_coef;
    pp.scale = &sc->scale;
    panel::dvp_panel_kernel<512, 2><<<(unsigned)rows, 512, 0, s>>>(pp);
    if (cudaGetLastError() != cudaSuccess) return DVP_ERR_CUDA;
    // d_hidden[r0 : r0 + rows] = diag(c) P W, the factor applied per row in the epilogue
    // few output tiles and a long K: two K ranges per tile fill the last wave of block pairs
    const long long dh_tiles = ((rows + 255) / 256) * (long long)((H + 255) / 256);
    e = gemm::launch_gemm_tn(p16, L.Vp, wt16, L.Vp, a->d_hidden + r0 * a->ld_dh, a->ld_dh, rows, H, V,
                             false, 1.f, nullptr, false, &sc->status, sms, s, false, false,
                             dh_tiles < 8LL * (sms / 2) ? 2 : 1, nullptr, 0, row_scale);
    if (e != cudaSuccess) return e == cudaErrorInvalidValue ? DVP_ERR_UNSUPPORTED : DVP_ERR_CUDA;
    // ... + q_t W[a_t]: the 1[k = a] term in fp32
    panel::add_sampled_rows_kernel<<<(unsigned)rows, 256, 0, s>>>(
        a->d_hidden + r0 * a->ld_dh, a->ld_dh, w, a->ld_w, p.ids, p.id_is_i32, a_coef, H);
    // the panel's hidden rows times their factor (and 2^14 * scale / 512), transposed, in float16
    launch_transpose<__nv_bfloat16, __half>(hidden + r0 * a->ld_hidden, a->ld_hidden, hs16, L.panel, rows, H, s,
                                            hid_scale);
    if (cudaGetLastError() != cudaSuccess) return DVP_ERR_CUDA;
    // d_w (+)= P^T x (scaled hidden rows) * 512 / (2^14 scale): P is read as it lies, [rows, V] with V
    // contiguous, as the transposed (MN-major) A operand of the contraction
    e = gemm::launch_gemm_tn(p16, L.Vp, hs16, L.panel, a->d_w, a->ld_dw, V, H, rows, false, 1.f / 32.f,
                             &sc->inv_scale, panel_index > 0 || a->accumulate_dw != 0, &sc->status, sms,
                             s, false, true);
    if (e != cudaSuccess) return e == cudaErrorInvalidValue ? DVP_ERR_UNSUPPORTED : DVP_ERR_CUDA;
    // ... + q_t hidden_t into row a_t of d_w: tokens that share a row are added in token order
    for (int c0 = 0; c0 < rows; c0 += panel::kSortChunk) {
      const int n = rows - c0 < panel::kSortChunk ? rows - c0 : panel::kSortChunk;
      const void *ids_c = static_cast<const char *>(p.ids) + (long long)c0 * id_bytes;
      panel::sort_sampled_ids_kernel<<<1, 1024, 0, s>>>(ids_c, p.id_is_i32, a_coef + c0, n, sorted);
      panel::add_sampled_hidden_kernel<<<panel::kSortChunk, 256, 0, s>>>(
          sorted, a_coef + c0, hidden + (r0 + c0) * a->ld_hidden, a->ld_hidden, a->d_w, a->ld_dw, H);
    }
    if (cudaGetLastError() != cudaSuccess) return DVP_ERR_CUDA;
  }

  if (a->infer_logits) {
    if (!weighted && infer_rows() != cudaSuccess) return DVP_ERR_CUDA;
    combine_sides_kernel<<<(unsigned)((a->T + 255) / 256), 256, 0, s>>>(a->T, lpt, lpi, fli, flt,
                                                                        a->log_ratio);
  }
  return cudaGetLastError() == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
}


// ---- a variant that allocates nothing ------------------------------------------
// The workspace of the fused entry point, taken from a fixed array that is part
// of the loaded library instead of from the caller.  In host code the array's
// name is only a handle; the device address comes from cudaGetSymbolAddress, once
// per device, with that device current.

}  // extern "C"

namespace {
constexpr size_t kStaticWorkspaceBytes = (size_t)DVP_STATIC_WORKSPACE_BYTES;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];
constexpr int kMaxDevices = 64;
void *g_static_workspace_ptr[kMaxDevices] = {};
std::mutex g_static_workspace_mutex;
}  // namespace

extern "C" {

int dvp_fused_lmhead_forward_backward_static(const dvp_fused_args *a) {
  if (!a || a->struct_size != sizeof(dvp_fused_args)) return DVP_ERR_INVALID_ARG;
  dvp_fused_args b = *a;
  if (b.panel_rows == 0) b.panel_rows = 128;  // the smallest panel leaves the most room
  dvp::FusedLayout L;
  if (!dvp::fused_layout(&b, &L)) return DVP_ERR_INVALID_ARG;
  if (L.total > kStaticWorkspaceBytes) return DVP_ERR_WORKSPACE;  // beyond the built-in maximum
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DVP_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return DVP_ERR_UNSUPPORTED;
  void *ptr = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_workspace_mutex);
    if (!g_static_workspace_ptr[dev]) {
      void *sym = nullptr;
      if (cudaGetSymbolAddress(&sym, g_static_workspace) != cudaSuccess || !sym) return DVP_ERR_CUDA;
      g_static_workspace_ptr[dev] = sym;
    }
    ptr = g_static_workspace_ptr[dev];
  }
  b.workspace = ptr;
  b.workspace_bytes = kStaticWorkspaceBytes;
  return dvp_fused_lmhead_forward_backward(&b);
}

int dvp_static_workspace_status(uint32_t *status_out) {
  if (!status_out) return DVP_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return DVP_ERR_CUDA;
  // the status is the first word of the workspace, here of the built-in array
  return cudaMemcpyFromSymbol(status_out, g_static_workspace, sizeof(uint32_t)) == cudaSuccess ? DVP_OK
                                                                                              : DVP_ERR_CUDA;
}

}  // extern "C"
