// Sequence-level aggregation of the per-token results and the token veto.
//
// The mismatch of a trajectory is the sum of its token mismatches (Sec. 4.4),
// its importance ratio the product of the token ratios (Thm. 5.3), and a token
// whose weight pi^mp_train / pi^mp_infer falls below the veto threshold discards
// the whole sequence (App. A, protocol 5).  One block per sequence, partial sums
// in double, fixed reduction order.
#include <cmath>

#include "dvp_common.cuh"

namespace dvp {

struct SeqPartial {
  double sum;
  double cov_sum;  // sum of the coverages Z_t = e^{ln Z_t}
  float lo;
  float cov_lo;
  int valid, zero, pinf, veto;
};

__device__ __forceinline__ SeqPartial seq_combine(const SeqPartial &a, const SeqPartial &b) {
  SeqPartial r;
  r.sum = a.sum + b.sum;
  r.cov_sum = a.cov_sum + b.cov_sum;
  r.lo = fminf(a.lo, b.lo);
  r.cov_lo = fminf(a.cov_lo, b.cov_lo);
  r.valid = a.valid + b.valid;
  r.zero = a.zero + b.zero;
  r.pinf = a.pinf | b.pinf;
  r.veto = a.veto | b.veto;
  return r;
}

__device__ __forceinline__ SeqPartial seq_shfl(const SeqPartial &v, int o) {
  SeqPartial r;
  r.sum = __shfl_xor_sync(0xffffffffu, v.sum, o);
  r.cov_sum = __shfl_xor_sync(0xffffffffu, v.cov_sum, o);
  r.lo = __shfl_xor_sync(0xffffffffu, v.lo, o);
  r.cov_lo = __shfl_xor_sync(0xffffffffu, v.cov_lo, o);
  r.valid = __shfl_xor_sync(0xffffffffu, v.valid, o);
  r.zero = __shfl_xor_sync(0xffffffffu, v.zero, o);
  r.pinf = __shfl_xor_sync(0xffffffffu, v.pinf, o);
  r.veto = __shfl_xor_sync(0xffffffffu, v.veto, o);
  return r;
}

__global__ void __launch_bounds__(256) dvp_sequence_kernel(const dvp_sequence_args a, float log_veto,
                                                           int veto_positive) {
  __shared__ SeqPartial part[8];
  const long long s = blockIdx.x;
  const long long t0 = a.seq_offsets[s], t1 = a.seq_offsets[s + 1];
  SeqPartial acc = {0.0, 0.0, -kNegInf, -kNegInf, 0, 0, 0, 0};
  // each thread takes a contiguous slice so that the order of the sum is fixed
  const long long n = t1 - t0, per = (n + blockDim.x - 1) / blockDim.x;
  const long long b = t0 + per * threadIdx.x, e = b + per < t1 ? b + per : t1;
  for (long long t = b; t < e; ++t) {
    if (a.log_cov) {  // the coverage of a state does not depend on the sampled token
      const float z = expf(a.log_cov[t]);
      acc.cov_sum += (double)z;
      acc.cov_lo = fminf(acc.cov_lo, z);
    }
    const float r = a.log_ratio[t];
    if (r != r) continue;  // no sampled token
    ++acc.valid;
    acc.lo = fminf(acc.lo, r);
    // weight e^r below the threshold: compared in the log domain, -inf always below a positive one
    if (veto_positive && r < log_veto) acc.veto = 1;
    if (r == kNegInf)
      ++acc.zero;
    else if (r == -kNegInf)
      acc.pinf = 1;
    else
      acc.sum += (double)r;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const SeqPartial other = seq_shfl(acc, o);
    acc = (lane & o) ? seq_combine(other, acc) : seq_combine(acc, other);
  }
  if (lane == 0) part[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    SeqPartial r = part[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = seq_combine(r, part[w]);
    if (a.seq_log_ratio)
      a.seq_log_ratio[s] = r.zero ? kNegInf : (r.pinf ? -kNegInf : (float)r.sum);
    if (a.min_log_ratio) a.min_log_ratio[s] = r.lo;
    if (a.n_valid) a.n_valid[s] = r.valid;
    if (a.n_zero_weight) a.n_zero_weight[s] = r.zero;
    if (a.veto) a.veto[s] = (uint8_t)r.veto;
    if (a.min_cov) a.min_cov[s] = r.cov_lo;
    if (a.mean_cov) a.mean_cov[s] = n > 0 ? (float)(r.cov_sum / (double)n) : __int_as_float(0x7fc00000);
  }
}

}  // namespace dvp

extern "C" int dvp_sequence_aggregate(const dvp_sequence_args *a) {
  if (!a || a->struct_size != sizeof(dvp_sequence_args)) return DVP_ERR_INVALID_ARG;
  if (a->S < 0 || a->S > 0x7fffffffLL || a->T < 0) return DVP_ERR_INVALID_ARG;
  if (!(a->veto_threshold >= 0.0)) return DVP_ERR_INVALID_ARG;
  if (a->S == 0) return DVP_OK;
  if (!a->seq_offsets || !a->log_ratio) return DVP_ERR_INVALID_ARG;
  if ((a->min_cov || a->mean_cov) && !a->log_cov) return DVP_ERR_INVALID_ARG;
  // e^r < threshold  <=>  r < ln(threshold).  With ln(threshold) rounded up to the next
  // float, "r < log_veto" decides every float r as the real-number comparison does.
  const int positive = a->veto_threshold > 0.0;
  float log_veto = 0.f;
  if (positive) {
    const double d = std::log(a->veto_threshold);
    log_veto = (float)d;
    if ((double)log_veto < d) log_veto = std::nextafterf(log_veto, HUGE_VALF);
  }
  dvp::dvp_sequence_kernel<<<(unsigned)a->S, 256, 0, static_cast<cudaStream_t>(a->stream)>>>(
      *a, log_veto, positive);
  return cudaGetLastError() == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
}
