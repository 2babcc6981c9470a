// Monitoring kernel: per-token Kullback-Leibler divergences between the
// full-vocabulary inference and training policies and their entropies (the
// stability metric of Sec. 6; the entropy Sec. 7 proposes to adapt rho to).
//
// Both rows are streamed together, once, in 32-byte granules.  Each thread keeps,
// for each policy, an online log-sum-exp state in the base-2 domain extended by
// two weighted sums: with w_k = 2^{z_k l - c},
//   s = sum w_k,  a = sum w_k z_k,  b = sum w_k (z'_k - z_k),
// from which  H = lse - a / s,  KL(train || infer) = -b/s - lse + lse',
// KL(infer || train) = b'/s' - lse' + lse.  HBM-bound: it reads both matrices once.
#include "dvp_rows_impl.cuh"

namespace dvp {

struct Moments {
  float m, c, s, a, b;
};

__device__ __forceinline__ Moments combine(const Moments &x, const Moments &y) {
  Moments r;
  r.m = fmaxf(x.m, y.m);
  r.c = fmaxf(x.c, y.c);
  const float fx = x.c > kNegInf ? ex2(x.c - r.c) : 0.f;
  const float fy = y.c > kNegInf ? ex2(y.c - r.c) : 0.f;
  r.s = x.s * fx + y.s * fy;
  r.a = x.a * fx + y.a * fy;
  r.b = x.b * fx + y.b * fy;
  return r;
}

__device__ __forceinline__ Moments shfl_xor(const Moments &v, int o) {
  Moments r;
  r.m = __shfl_xor_sync(0xffffffffu, v.m, o);
  r.c = __shfl_xor_sync(0xffffffffu, v.c, o);
  r.s = __shfl_xor_sync(0xffffffffu, v.s, o);
  r.a = __shfl_xor_sync(0xffffffffu, v.a, o);
  r.b = __shfl_xor_sync(0xffffffffu, v.b, o);
  return r;
}

// scratch: 5 x 32 floats.  Fixed order; the result is valid in every thread.
__device__ __forceinline__ Moments block_reduce(Moments v, float *scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const Moments other = shfl_xor(v, o);
    v = (lane & o) ? combine(other, v) : combine(v, other);
  }
  __syncthreads();
  if (lane == 0) {
    scratch[warp] = v.m;
    scratch[32 + warp] = v.c;
    scratch[64 + warp] = v.s;
    scratch[96 + warp] = v.a;
    scratch[128 + warp] = v.b;
  }
  __syncthreads();
  Moments r = {kNegInf, kNegInf, 0.f, 0.f, 0.f};
  if (lane < nwarp) {
    r.m = scratch[lane];
    r.c = scratch[32 + lane];
    r.s = scratch[64 + lane];
    r.a = scratch[96 + lane];
    r.b = scratch[128 + lane];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const Moments other = shfl_xor(r, o);
    r = (lane & o) ? combine(other, r) : combine(r, other);
  }
  return r;
}

// Move the reference of a state to a larger maximum.
__device__ __forceinline__ void raise(Moments &v, float new_max) {
  if (new_max > v.m) {
    const float cn = new_max * kLog2e;
    const float f = ex2(v.c - cn);  // v.c = -inf at the start: factor 0
    v.s *= f;
    v.a *= f;
    v.b *= f;
    v.m = new_max;
    v.c = cn;
  }
}

__device__ __forceinline__ void absorb(Moments &v, float x, float d) {
  const float w = ex2(fmaf(x, kLog2e, -v.c));
  v.s += w;
  v.a = fmaf(w, x, v.a);
  v.b = fmaf(w, d, v.b);
}

struct MonitorParams {
  const void *train, *infer;
  long long T, V, ld_train, ld_infer;
  float *kl_it, *kl_ti, *h_t, *h_i;
  unsigned int *bounds_status;  // the bounds-checking build's status word; unused otherwise
};

__device__ __forceinline__ void monitor_finish(const MonitorParams &p, long long t, const Moments &a,
                                               const Moments &b) {
  const double ln2 = 0.6931471805599453094;
  const double corr = 1.0 - (double)kLog2e * ln2;
  const double lse_t = ln2 * ((double)a.c + (double)log2f(a.s)) + corr * (double)a.m;
  const double lse_i = ln2 * ((double)b.c + (double)log2f(b.s)) + corr * (double)b.m;
  const double ez_t = (double)a.a / (double)a.s, ed_t = (double)a.b / (double)a.s;
  const double ez_i = (double)b.a / (double)b.s, ed_i = (double)b.b / (double)b.s;
  if (p.kl_ti) p.kl_ti[t] = (float)(-ed_t - lse_t + lse_i);
  if (p.kl_it) p.kl_it[t] = (float)(ed_i - lse_i + lse_t);
  if (p.h_t) p.h_t[t] = (float)(lse_t - ez_t);
  if (p.h_i) p.h_i[t] = (float)(lse_i - ez_i);
}

template <typename TIn, bool kVector>
__global__ void __launch_bounds__(256, 3) dvp_monitor_kernel(const MonitorParams p) {
  __shared__ float scratch[160];
  constexpr int kElems = Granule<TIn>::kElems;
  const long long t = blockIdx.x;
  const TIn *zt = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
  const TIn *zi = reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer;
  const int V = (int)p.V;
  DVP_BOUNDS_BEGIN(p.bounds_status);
  DVP_BOUNDS_SET(n_gran, (V + kElems - 1) / kElems);
  DVP_BOUNDS_SET(V, V);
  DVP_BOUNDS_SYNC();
  Moments a = {kNegInf, kNegInf, 0.f, 0.f, 0.f}, b = a;
  if constexpr (kVector) {
    // whole granules in the loop; the elements behind the last whole granule one per thread after
    // it, so that the loop carries no element-wise code for a ragged granule
    const int n_full = V / kElems;
    for (int g = threadIdx.x; g < n_full; g += 2 * blockDim.x) {
      const int g2 = g + blockDim.x;
      Granule<TIn> ta, ia, tb, ib;  // two granules of each row in flight
      if (!DVP_IN((long long)g * kElems + kElems - 1, V, DVP_OOB_GLOBAL)) break;
      ta.load(zt + (size_t)g * kElems);
      ia.load(zi + (size_t)g * kElems);
      const bool second = g2 < n_full && DVP_IN((long long)g2 * kElems + kElems - 1, V, DVP_OOB_GLOBAL);
      if (second) {
        tb.load(zt + (size_t)g2 * kElems);
        ib.load(zi + (size_t)g2 * kElems);
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h == 1 && !second) break;
        const Granule<TIn> &gt = h ? tb : ta, &gi = h ? ib : ia;
        float x[kElems], y[kElems];
        gt.get(x);
        gi.get(y);
        raise(a, gt.max());
        raise(b, gi.max());
#pragma unroll
        for (int j = 0; j < kElems; ++j) {
          const float d = y[j] - x[j];
          absorb(a, x[j], d);
          absorb(b, y[j], d);
        }
      }
    }
    const int k_tail = n_full * kElems + (int)threadIdx.x;
    if (k_tail < V) {
      const float x = Storage<TIn>::widen(zt[k_tail]), y = Storage<TIn>::widen(zi[k_tail]);
      raise(a, x);
      raise(b, y);
      absorb(a, x, y - x);
      absorb(b, y, y - x);
    }
  } else {
    float mt = kNegInf, mi = kNegInf;
    for (long long k = threadIdx.x; k < p.V; k += blockDim.x) {
      mt = fmaxf(mt, Storage<TIn>::widen(zt[k]));
      mi = fmaxf(mi, Storage<TIn>::widen(zi[k]));
    }
    raise(a, mt);
    raise(b, mi);
    for (long long k = threadIdx.x; k < p.V; k += blockDim.x) {
      const float x = Storage<TIn>::widen(zt[k]), y = Storage<TIn>::widen(zi[k]);
      absorb(a, x, y - x);
      absorb(b, y, y - x);
    }
  }
  const Moments ra = block_reduce(a, scratch);
  const Moments rb = block_reduce(b, scratch);
  if (threadIdx.x == 0) monitor_finish(p, t, ra, rb);
}

template <typename TIn>
static cudaError_t launch_monitor(const MonitorParams &p, cudaStream_t s) {
  const bool vec = aligned32(p.train, p.ld_train, sizeof(TIn)) && aligned32(p.infer, p.ld_infer, sizeof(TIn));
  if (vec)
    dvp_monitor_kernel<TIn, true><<<(unsigned)p.T, 256, 0, s>>>(p);
  else
    dvp_monitor_kernel<TIn, false><<<(unsigned)p.T, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace dvp

extern "C" int dvp_monitor(const dvp_monitor_args *a) {
  if (!a || a->struct_size != sizeof(dvp_monitor_args)) return DVP_ERR_INVALID_ARG;
  if (a->logits_dtype != DVP_F32 && a->logits_dtype != DVP_BF16 && a->logits_dtype != DVP_F16)
    return DVP_ERR_UNSUPPORTED;
  if (a->T < 0 || a->T > 0x7fffffffLL || a->V < 1) return DVP_ERR_INVALID_ARG;
  if (a->V > 0x7fffff00LL) return DVP_ERR_UNSUPPORTED;
  if (a->T == 0) return DVP_OK;
  if (!a->train_logits || !a->infer_logits || a->ld_train < a->V || a->ld_infer < a->V)
    return DVP_ERR_INVALID_ARG;
  dvp::MonitorParams p{a->train_logits, a->infer_logits, a->T, a->V, a->ld_train, a->ld_infer,
                       a->kl_infer_train, a->kl_train_infer, a->entropy_train, a->entropy_infer,
                       dvp::bounds_status_word()};
  cudaStream_t s = static_cast<cudaStream_t>(a->stream);
  cudaError_t e;
  switch (a->logits_dtype) {
    case DVP_F32: e = dvp::launch_monitor<float>(p, s); break;
    case DVP_BF16: e = dvp::launch_monitor<__nv_bfloat16>(p, s); break;
    default: e = dvp::launch_monitor<__half>(p, s); break;
  }
  return e == cudaSuccess ? DVP_OK : DVP_ERR_CUDA;
}
