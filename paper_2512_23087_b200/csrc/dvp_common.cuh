// Shared device helpers of the DVP row kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dvp.h"

namespace dvp {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegInf = -__builtin_huge_valf();

// e^{x} for x already multiplied by log2(e): one MUFU op, flushes denormals.
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- bounds-checking build (-DDVP_DEBUG_BOUNDS) ------------------------------------
// Stands in for a memory checker: every shared-memory index of the row kernels' tables
// (granule bounds, hot lists, candidate rings and lists, resident slots) and every global
// element offset they form is compared with its extent.  An index out of range is not
// used: the access is skipped and a code is OR-ed into a per-device status word that
// dvp_debug_bounds_status reads.  Nothing traps.  In the ordinary build the checks
// compile to nothing.
enum : unsigned {
  DVP_OOB_BOUND = 1,    // granule-bound table
  DVP_OOB_HOT = 2,      // hot-list entry
  DVP_OOB_GRANULE = 4,  // granule index outside the row
  DVP_OOB_GLOBAL = 8,   // global element offset outside the row
  DVP_OOB_RING = 16,    // candidate ring slot
  DVP_OOB_LIST = 32,    // candidate list entry
  DVP_OOB_SLOT = 64     // resident-row slot or its bytes
};
#ifdef DVP_DEBUG_BOUNDS
struct BoundsCtx {
  unsigned int *status;
  long long n_bound, n_hot, n_gran, V, n_ring, n_list, n_slot;
};
// one instance per block (a __shared__ variable of a device function)
__device__ __forceinline__ BoundsCtx &bounds_ctx() {
  __shared__ BoundsCtx c;
  return c;
}
__device__ __forceinline__ bool bounds_ok(long long i, long long n, unsigned code) {
  if (i >= 0 && i < n) return true;
  if (bounds_ctx().status) atomicOr(bounds_ctx().status, code);
  return false;
}
#define DVP_IN(i, field, code) ::dvp::bounds_ok((long long)(i), ::dvp::bounds_ctx().field, code)
#define DVP_BOUNDS_SET(field, value) \
  do { if (threadIdx.x == 0) ::dvp::bounds_ctx().field = (value); } while (0)
#define DVP_BOUNDS_BEGIN(ptr)                                                                    \
  do {                                                                                           \
    if (threadIdx.x == 0) {                                                                      \
      ::dvp::BoundsCtx &c_ = ::dvp::bounds_ctx();                                                \
      c_.status = (ptr);                                                                         \
      c_.n_bound = c_.n_hot = c_.n_gran = c_.V = c_.n_ring = c_.n_list = c_.n_slot = 0;                     \
    }                                                                                            \
    __syncthreads();                                                                             \
  } while (0)
#define DVP_BOUNDS_SYNC() __syncthreads()
#else
#define DVP_IN(i, field, code) true
#define DVP_BOUNDS_SET(field, value) do { } while (0)
#define DVP_BOUNDS_BEGIN(ptr) do { } while (0)
#define DVP_BOUNDS_SYNC() do { } while (0)
#endif

// 16-byte read-only load that does not allocate in L1: each logit is consumed
// once per sweep, re-reads are served by L2.
__device__ __forceinline__ uint4 ld_stream16(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// 32-byte variant: one DRAM sector per lane and instruction.
__device__ __forceinline__ void ld_stream32(const void *p, uint32_t (&w)[8]) {
  asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]),
                 "=r"(w[7])
               : "l"(p));
}

// Streaming stores (evict-first): the gradient is written once and not read
// again by this library.
__device__ __forceinline__ void st_stream16(void *p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}
__device__ __forceinline__ void st_stream32(void *p, const uint32_t (&w)[8]) {
  asm volatile("st.global.cs.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]),
               "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}
__device__ __forceinline__ void st_stream8(void *p, uint2 v) {
  asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
}

// ---- storage types ---------------------------------------------------------

template <typename T>
struct Storage;

template <>
struct Storage<float> {
  static constexpr int kPerVec = 4;  // elements in 16 bytes
  static __device__ __forceinline__ void unpack(uint4 r, float *x) {
    x[0] = __uint_as_float(r.x);
    x[1] = __uint_as_float(r.y);
    x[2] = __uint_as_float(r.z);
    x[3] = __uint_as_float(r.w);
  }
  static __device__ __forceinline__ float widen(float v) { return v; }
  static __device__ __forceinline__ float narrow(float v) { return v; }
};

template <>
struct Storage<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  static __device__ __forceinline__ void unpack(uint4 r, float *x) {
    // a bfloat16 is the upper half of a binary32
    x[0] = __uint_as_float(r.x << 16);
    x[1] = __uint_as_float(r.x & 0xffff0000u);
    x[2] = __uint_as_float(r.y << 16);
    x[3] = __uint_as_float(r.y & 0xffff0000u);
    x[4] = __uint_as_float(r.z << 16);
    x[5] = __uint_as_float(r.z & 0xffff0000u);
    x[6] = __uint_as_float(r.w << 16);
    x[7] = __uint_as_float(r.w & 0xffff0000u);
  }
  static __device__ __forceinline__ float widen(__nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ __forceinline__ __nv_bfloat16 narrow(float v) { return __float2bfloat16_rn(v); }
};

template <>
struct Storage<__half> {
  static constexpr int kPerVec = 8;
  static __device__ __forceinline__ void unpack(uint4 r, float *x) {
    const __half2 *h = reinterpret_cast<const __half2 *>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __half22float2(h[i]);
      x[2 * i] = f.x;
      x[2 * i + 1] = f.y;
    }
  }
  static __device__ __forceinline__ float widen(__half v) { return __half2float(v); }
  static __device__ __forceinline__ __half narrow(float v) { return __float2half_rn(v); }
};

// Store N consecutive gradients (N = 4 or 8), round-to-nearest-even, to an
// address aligned to N * sizeof(TG).
template <typename TG, int N>
__device__ __forceinline__ void store_grads(TG *dst, const float *g) {
  if constexpr (sizeof(TG) == 4) {
#pragma unroll
    for (int i = 0; i < N; i += 4)
      st_stream16(dst + i, make_uint4(__float_as_uint(g[i]), __float_as_uint(g[i + 1]),
                                      __float_as_uint(g[i + 2]), __float_as_uint(g[i + 3])));
  } else {
    uint32_t w[N / 2];
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      TG lo = Storage<TG>::narrow(g[2 * i]), hi = Storage<TG>::narrow(g[2 * i + 1]);
      w[i] = (uint32_t) * reinterpret_cast<uint16_t *>(&lo) |
             ((uint32_t) * reinterpret_cast<uint16_t *>(&hi) << 16);
    }
    if constexpr (N == 8)
      st_stream16(dst, make_uint4(w[0], w[1], w[2], w[3]));
    else
      st_stream8(dst, make_uint2(w[0], w[1]));
  }
}

template <typename TG, int N>
__device__ __forceinline__ void store_zeros(TG *dst) {
  if constexpr (sizeof(TG) == 4) {
#pragma unroll
    for (int i = 0; i < N; i += 4) st_stream16(dst + i, make_uint4(0, 0, 0, 0));
  } else if constexpr (N == 8) {
    st_stream16(dst, make_uint4(0, 0, 0, 0));
  } else {
    st_stream8(dst, make_uint2(0, 0));
  }
}

// ---- block reductions in a fixed order (bit-identical from run to run) ------

// Partial log-sum-exp state: sum of e^{z - m} over the elements seen so far.
struct MaxSum {
  float m, s;
};

__device__ __forceinline__ MaxSum combine(MaxSum a, MaxSum b) {
  const float m = fmaxf(a.m, b.m);
  MaxSum r;
  r.m = m;
  // a side that has seen nothing carries m = -inf and contributes nothing
  const float sa = a.m > kNegInf ? a.s * ex2((a.m - m) * kLog2e) : 0.f;
  const float sb = b.m > kNegInf ? b.s * ex2((b.m - m) * kLog2e) : 0.f;
  r.s = sa + sb;
  return r;
}

// scratch: 64 floats of shared memory.  Result valid in every thread.
__device__ __forceinline__ MaxSum block_reduce_maxsum(MaxSum v, float *scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    MaxSum other;
    other.m = __shfl_xor_sync(0xffffffffu, v.m, o);
    other.s = __shfl_xor_sync(0xffffffffu, v.s, o);
    // keep operand order independent of the lane so both partners agree
    v = (lane & o) ? combine(other, v) : combine(v, other);
  }
  __syncthreads();  // scratch may still be read from an earlier reduction
  if (lane == 0) {
    scratch[warp] = v.m;
    scratch[32 + warp] = v.s;
  }
  __syncthreads();
  MaxSum r;
  r.m = lane < nwarp ? scratch[lane] : kNegInf;
  r.s = lane < nwarp ? scratch[32 + lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    MaxSum other;
    other.m = __shfl_xor_sync(0xffffffffu, r.m, o);
    other.s = __shfl_xor_sync(0xffffffffu, r.s, o);
    r = (lane & o) ? combine(other, r) : combine(r, other);
  }
  return r;
}

// Log-sum-exp state kept in the base-2 domain so that each term costs one FMA
// and one ex2: with l = kLog2e (a float), the elements seen so far satisfy
//   sum_k 2^{z_k l} = 2^c s,   c = fl(m l),   m = their maximum.
struct LogSum {
  float m, c, s;
};

__device__ __forceinline__ LogSum combine(LogSum a, LogSum b) {
  LogSum r;
  r.m = fmaxf(a.m, b.m);
  r.c = fmaxf(a.c, b.c);
  const float sa = a.c > kNegInf ? a.s * ex2(a.c - r.c) : 0.f;
  const float sb = b.c > kNegInf ? b.s * ex2(b.c - r.c) : 0.f;
  r.s = sa + sb;
  return r;
}

// scratch: 96 floats of shared memory.  Result valid in every thread.
__device__ __forceinline__ LogSum block_reduce_logsum(LogSum v, float *scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    LogSum other;
    other.m = __shfl_xor_sync(0xffffffffu, v.m, o);
    other.c = __shfl_xor_sync(0xffffffffu, v.c, o);
    other.s = __shfl_xor_sync(0xffffffffu, v.s, o);
    v = (lane & o) ? combine(other, v) : combine(v, other);
  }
  __syncthreads();
  if (lane == 0) {
    scratch[warp] = v.m;
    scratch[32 + warp] = v.c;
    scratch[64 + warp] = v.s;
  }
  __syncthreads();
  LogSum r;
  r.m = lane < nwarp ? scratch[lane] : kNegInf;
  r.c = lane < nwarp ? scratch[32 + lane] : kNegInf;
  r.s = lane < nwarp ? scratch[64 + lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    LogSum other;
    other.m = __shfl_xor_sync(0xffffffffu, r.m, o);
    other.c = __shfl_xor_sync(0xffffffffu, r.c, o);
    other.s = __shfl_xor_sync(0xffffffffu, r.s, o);
    r = (lane & o) ? combine(other, r) : combine(r, other);
  }
  return r;
}

// ln sum_k e^{z_k} from the base-2 state.  2^{z l} = e^{z lambda} with
// lambda = l ln 2 = 1 - 1.3e-8, so ln sum e^{z} = ln 2 (c + log2 s) +
// (1 - lambda) E[z], the mean taken under the softmax weights; the maximum
// stands in for it (they differ by at most about ln V, times 1.3e-8).
__device__ __forceinline__ double lse_from_logsum(const LogSum &v) {
  const double ln2 = 0.6931471805599453094;
  const double one_minus_lambda = 1.0 - (double)kLog2e * ln2;
  return ln2 * ((double)v.c + (double)log2f(v.s)) + one_minus_lambda * (double)v.m;
}

struct SumCount {
  float s;
  int n;
};

__device__ __forceinline__ SumCount block_reduce_sumcount(SumCount v, float *scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float os = __shfl_xor_sync(0xffffffffu, v.s, o);
    const int on = __shfl_xor_sync(0xffffffffu, v.n, o);
    v.s = (lane & o) ? os + v.s : v.s + os;
    v.n += on;
  }
  __syncthreads();
  if (lane == 0) {
    scratch[warp] = v.s;
    reinterpret_cast<int *>(scratch)[32 + warp] = v.n;
  }
  __syncthreads();
  SumCount r;
  r.s = lane < nwarp ? scratch[lane] : 0.f;
  r.n = lane < nwarp ? reinterpret_cast<int *>(scratch)[32 + lane] : 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float os = __shfl_xor_sync(0xffffffffu, r.s, o);
    const int on = __shfl_xor_sync(0xffffffffu, r.n, o);
    r.s = (lane & o) ? os + r.s : r.s + os;
    r.n += on;
  }
  return r;
}

// Maximum over the block.  scratch: 32 floats.  Result valid in every thread.
__device__ __forceinline__ float block_reduce_max(float v, float *scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float r = lane < nwarp ? scratch[lane] : kNegInf;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, o));
  return r;
}

// ---- per-row bookkeeping shared by all row kernels ---------------------------

struct RowParams {
  const void *train, *infer, *ids;
  const float *upstream;
  void *grad;
  long long T, V, ld_train, ld_infer, ld_grad;
  double log_rho;  // ln(rho); -inf for rho = 0
  int id_is_i32;
  int mode;          // DVP_MODE_* bits
  float mask_value;  // finite mask value (DVP_MODE_FINITE_MASK)
  dvp_side_out out_t, out_i;
  float *log_ratio;
  uint8_t *flags;
  int weight_kind;  // DVP_WEIGHT_*: the upstream gradient is multiplied by the token's importance weight
  float weight_lo, weight_hi;
  float *weight_out;
  // the inference side of the weight when an earlier launch computed it (no `infer` matrix then):
  // ln pi^mp_infer(a) per token, and flags whose DVP_FLAG_IN_TRAIN bit says "a in V'_S"
  const float *given_logp_mp_i;
  const uint8_t *given_flags_i;
  unsigned int *bounds_status;  // the bounds-checking build's status word; unused otherwise
};

__device__ __forceinline__ long long load_id(const void *ids, int is_i32, long long t) {
  return is_i32 ? (long long)reinterpret_cast<const int *>(ids)[t]
                : reinterpret_cast<const long long *>(ids)[t];
}

// Threshold in the logits' own precision: the smallest float that is >= the
// double m + ln(rho).  For stored values that are floats (or narrower),
// "z >= tau_f" then decides exactly as the double comparison does.
__device__ __forceinline__ float threshold_f32(float m, double log_rho) {
  return __double2float_ru((double)m + log_rho);
}

// The threshold as an eager tensor expression of the logits' type forms it
// (DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE), or the exact one.
template <typename TIn>
__device__ __forceinline__ float threshold_of(float m, double log_rho, int mode) {
  if (mode & DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE) {
    const float c = Storage<TIn>::widen(Storage<TIn>::narrow((float)log_rho));
    return Storage<TIn>::widen(Storage<TIn>::narrow(m + c));
  }
  return threshold_f32(m, log_rho);
}

// Everything one side of one row reduces to.
struct SideStats {
  float m;       // row max
  double lse;    // ln sum_k e^{z_k}
  double sum_c;  // the full sum as 2^sum_c * sum_s (base 2, exponents scaled by kLog2e as the safe sum is)
  float sum_s;
  float s_x;     // sum over the safe set of e^{z_k - m}, without the sampled token
  float e_a;     // e^{z_a - m} when a is in the safe set, else 0
  float s_mask;  // mass of the masked tokens, (V - n) e^{mask_value - m}; 0 without a finite mask
  float e_mask;  // e^{mask_value - m}; 0 without a finite mask
  float z_a;     // logit of the sampled token (0 when there is none)
  float tau;     // threshold
  int n;         // |V_S|
  int member;    // a in V_S
  int live;      // the row has a gradient: a valid and (a in V_S or finite mask)
};

// Mass of the masked tokens once the count is known.
__device__ __forceinline__ void set_mask_mass(SideStats &st, long long V, int mode, float mask_value_d,
                                              bool has_a) {
  st.e_mask = (mode & DVP_MODE_FINITE_MASK) ? ex2((mask_value_d - st.m) * kLog2e) : 0.f;
  st.s_mask = (float)(V - st.n) * st.e_mask;
  st.live = has_a && (st.member || (mode & DVP_MODE_FINITE_MASK));
}

// ln pi^mp(a) of a row with a valid sampled token, with the arithmetic of finish_side.
__device__ __forceinline__ float logp_mp_of(const SideStats &st) {
  const float log_ss = logf(st.s_x + st.e_a + st.s_mask);
  if (st.member) return (st.z_a - st.m) - log_ss;
  if (st.e_mask > 0.f) return logf(st.e_mask) - log_ss;  // a masked token keeps the mask value's probability
  return kNegInf;
}

// Writes the per-token outputs of one side; called by one thread.
__device__ __forceinline__ float finish_side(const dvp_side_out &o, long long t, const SideStats &st,
                                             bool has_id, bool bad_id) {
  const float s_tot = st.s_x + st.e_a + st.s_mask;
  const float log_ss = logf(s_tot);
  const float nan = __int_as_float(0x7fc00000);
  float logp = nan, logp_mp = nan, comp = nan;
  if (has_id) {
    logp = (float)((double)st.z_a - st.lse);
    if (st.member) {
      logp_mp = (st.z_a - st.m) - log_ss;
      comp = (st.s_x + st.s_mask) / s_tot;
    } else if (st.e_mask > 0.f) {  // a masked token keeps the mask value's probability
      logp_mp = logf(st.e_mask) - log_ss;
      comp = (s_tot - st.e_mask) / s_tot;
    } else {
      logp_mp = kNegInf;
      comp = 1.f;
    }
  }
  if (bad_id) logp = logp_mp = comp = nan;
  if (o.max) o.max[t] = st.m;
  if (o.lse) o.lse[t] = (float)st.lse;
  if (o.lse_safe) o.lse_safe[t] = st.m + log_ss;
  if (o.logp) o.logp[t] = logp;
  if (o.logp_mp) o.logp_mp[t] = logp_mp;
  if (o.comp_mp) o.comp_mp[t] = comp;
  if (o.count) o.count[t] = st.n;
  if (o.log_cov) {
    // ln Z = ln(safe sum / full sum), both sums of 2^{z l}; one thread, so double logarithms cost nothing
    const double safe2 = (double)st.m * (double)kLog2e + log2((double)st.s_x + (double)st.e_a);
    const double full2 = st.sum_c + log2((double)st.sum_s);
    o.log_cov[t] = (float)fmin(0.0, 0.6931471805599453094 * (safe2 - full2));
  }
  return logp_mp;
}

// ln pi^mp_train(a) - ln pi^mp_infer(a) with the conventions for pruned tokens.
__device__ __forceinline__ float log_ratio_of(bool in_train, bool in_infer, float lt, float li) {
  if (!in_train) return kNegInf;
  if (!in_infer) return -kNegInf;
  return lt - li;
}

// Token-level importance weight from the log-ratio r (DVP_WEIGHT_*): the per-token
// factor of the estimator of Thm. 5.3, optionally truncated or masked.
__device__ __forceinline__ float token_weight(float r, int kind, float lo, float hi) {
  if (kind == DVP_WEIGHT_NONE) return 1.f;
  if (r != r) return r;
  const float w = expf(r);  // e^{-inf} = 0, e^{+inf} = +inf
  if (kind == DVP_WEIGHT_RATIO) return w;
  if (kind == DVP_WEIGHT_TRUNCATE) return fminf(w, hi);
  return (w >= lo && w <= hi) ? w : 0.f;
}

// The weight of row t from the statistics of both sides (every thread computes the
// same value), NaN without a valid sampled token.
__device__ __forceinline__ float row_weight(const RowParams &p, const SideStats &st, const SideStats &si,
                                            bool valid_id) {
  if (!valid_id) return __int_as_float(0x7fc00000);
  const float lt = logp_mp_of(st), li = logp_mp_of(si);
  const float r = (p.mode & DVP_MODE_FINITE_MASK) ? lt - li : log_ratio_of(st.member, si.member, lt, li);
  return token_weight(r, p.weight_kind, p.weight_lo, p.weight_hi);
}

// The same from an inference side computed by an earlier launch.
__device__ __forceinline__ float row_weight_given(const RowParams &p, const SideStats &st, long long t,
                                                  bool valid_id) {
  if (!valid_id) return __int_as_float(0x7fc00000);
  const float lt = logp_mp_of(st), li = p.given_logp_mp_i[t];
  const bool in_i = (p.given_flags_i[t] & DVP_FLAG_IN_TRAIN) != 0;
  return token_weight(log_ratio_of(st.member, in_i, lt, li), p.weight_kind, p.weight_lo, p.weight_hi);
}

// Arguments of the stand-alone backward map.
struct BackwardParams {
  const void *train, *ids;
  const float *upstream, *max_t, *lse_safe_t, *comp_mp_t;
  const uint8_t *flags;
  void *grad;
  long long T, V, ld_train, ld_grad;
  double log_rho;
  int id_is_i32;
  int mode;
  float mask_value;
  unsigned int *bounds_status;  // the bounds-checking build's status word; unused otherwise
};

// Launchers (dvp_rows.cu).  `hint`: threads per block in the low 16 bits,
// 32-byte loads per thread and pipeline stage in the next 8 bits, 0 = default.
cudaError_t launch_row_kernels(const RowParams &p, int logits_dtype, int grad_dtype, uint32_t hint,
                               cudaStream_t s);
cudaError_t launch_backward_kernel(const BackwardParams &p, int logits_dtype, int grad_dtype,
                                   uint32_t hint, cudaStream_t s);

// Synchronises the current device, reads the resident-row kernel's status word and clears it.
cudaError_t read_and_clear_row_status(uint32_t *host_out);

// Device address of the bounds-checking build's status word (nullptr in the ordinary build),
// and its value after a device synchronisation (cleared by the read).
unsigned int *bounds_status_word();
cudaError_t read_and_clear_bounds_status(uint32_t *host_out);

}  // namespace dvp
