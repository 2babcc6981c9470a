// Row kernels of Dynamic Vocabulary Pruning for sm_100a.
//
// One thread block owns one token row.  The row is streamed from HBM once
// (sweep 1).  While it streams, every thread keeps an online log-sum-exp of
// what it has seen and leaves in shared memory the maximum of each chunk it
// loaded (a chunk = kUnroll 16-byte vectors of one thread).  Once the row
// maximum, hence the threshold of Def. 5.1, is known, only the chunks whose
// maximum reaches the threshold can hold safe tokens: sweep 2 (masked sum and
// count, Def. 5.2) and sweep 3 (gradient, Prop. 5.4) revisit just those,
// normally out of L2, and sweep 3 writes zeros for all the others without
// reading anything.  With a sparse safe set the row costs one HBM read per
// logit matrix and one HBM write of the gradient; with a dense safe set the
// same code degrades to three sweeps, still correct.
#include "dvp_common.cuh"

namespace dvp {

// A chunk: the kUnroll 16-byte vectors that thread `tid` loads in sweep step
// `i`, vector u at index (i * kUnroll + u) * blockDim + tid, kept packed as
// loaded.  Elements past V are filled with -inf.
template <typename TIn, int kUnroll>
struct Chunk {
  static constexpr int kPerVec = Storage<TIn>::kPerVec;
  uint4 raw[kUnroll];

  __device__ __forceinline__ void load(const TIn *row, int V, int n_full, int vb, int tid) {
    const int v0 = vb + tid;
    if (vb + kUnroll * (int)blockDim.x <= n_full) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u)
        raw[u] = ld_stream16(row + (size_t)(v0 + u * (int)blockDim.x) * kPerVec);
    } else {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int v = v0 + u * (int)blockDim.x;
        if (v < n_full) {
          raw[u] = ld_stream16(row + (size_t)v * kPerVec);
        } else {
          __align__(16) TIn tmp[kPerVec];
#pragma unroll
          for (int j = 0; j < kPerVec; ++j) {
            const long long k = (long long)v * kPerVec + j;
            tmp[j] = k < V ? row[k] : Storage<TIn>::narrow(kNegInf);
          }
          raw[u] = *reinterpret_cast<const uint4 *>(tmp);
        }
      }
    }
  }

  __device__ __forceinline__ void get(int u, float *x) const { Storage<TIn>::unpack(raw[u], x); }
};

// Chunks that can hold a safe token, per warp, in the order (sweep step, lane).
// A warp whose chunks do not fit (a dense safe set) walks all of its chunks
// instead, which is then the efficient thing to do anyway.
constexpr int kHotCap = 128;

struct HotList {
  uint32_t *slots;  // kHotCap entries of this warp: step * 32 + lane
  int count;        // chunks at or above the threshold (may exceed kHotCap)
  __device__ __forceinline__ bool fits() const { return count <= kHotCap; }
};

__device__ __forceinline__ HotList build_hot_list(const float *chunk_max, int n_steps, float tau,
                                                  uint32_t *hot_smem) {
  const int lane = threadIdx.x & 31;
  HotList h;
  h.slots = hot_smem + (threadIdx.x >> 5) * kHotCap;
  h.count = 0;
  for (int i = 0; i < n_steps; ++i) {
    const bool f = chunk_max[i * blockDim.x + threadIdx.x] >= tau;
    const unsigned b = __ballot_sync(0xffffffffu, f);
    if (f) {
      const int pos = h.count + __popc(b & ((1u << lane) - 1u));
      if (pos < kHotCap) h.slots[pos] = (uint32_t)(i * 32 + lane);
    }
    h.count += __popc(b);
  }
  __syncwarp();
  return h;
}

// Contribution of one chunk to the masked sum and the count (Def. 5.2).
template <typename TIn, int kUnroll>
__device__ __forceinline__ void chunk_masked_sum(const Chunk<TIn, kUnroll> &c, int vb, int tid,
                                                 int a, int va, float tau, float m, SumCount &sc) {
  constexpr int kPerVec = Storage<TIn>::kPerVec;
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    const int v = vb + u * (int)blockDim.x + tid;
    float x[kPerVec];
    c.get(u, x);
    // the sampled token is left out so that 1 - pi^mp(a) has no cancellation
    const int ja = v == va ? a - va * kPerVec : -1;
#pragma unroll
    for (int j = 0; j < kPerVec; ++j) {
      if (x[j] >= tau) {
        ++sc.n;
        if (j != ja) sc.s += ex2((x[j] - m) * kLog2e);
      }
    }
  }
}

// Sweeps 1 and 2 over one row: statistics of one side.
template <typename TIn, int kUnroll>
__device__ __forceinline__ SideStats row_stats(const TIn *row, int V, int a, double log_rho,
                                               float *chunk_max, float *scratch, uint32_t *hot_smem,
                                               HotList &hot, uint32_t *mask_row) {
  constexpr int kPerVec = Storage<TIn>::kPerVec;
  const int n_full = V / kPerVec;
  const int n_vec = (V + kPerVec - 1) / kPerVec;
  const int per_sweep = kUnroll * (int)blockDim.x;
  const int n_steps = (n_vec + per_sweep - 1) / per_sweep;
  const int tid = threadIdx.x;

  // ---- sweep 1: online max / sum-exp, chunk maxima to shared memory
  MaxSum acc = {kNegInf, 0.f};
  for (int i = 0; i < n_steps; ++i) {
    Chunk<TIn, kUnroll> c;
    c.load(row, V, n_full, i * per_sweep, tid);
    float cm = kNegInf;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float x[kPerVec];
      c.get(u, x);
#pragma unroll
      for (int j = 0; j < kPerVec; ++j) cm = fmaxf(cm, x[j]);
    }
    chunk_max[i * blockDim.x + tid] = cm;
    if (cm > kNegInf) {
      if (cm > acc.m) {
        acc.s *= ex2((acc.m - cm) * kLog2e);
        acc.m = cm;
      }
      float part = 0.f;
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        float x[kPerVec];
        c.get(u, x);
#pragma unroll
        for (int j = 0; j < kPerVec; ++j) part += ex2((x[j] - acc.m) * kLog2e);
      }
      acc.s += part;
    }
  }
  const MaxSum all = block_reduce_maxsum(acc, scratch);

  SideStats st;
  st.m = all.m;
  st.s = all.s;
  st.tau = threshold_f32(all.m, log_rho);
  const bool has_a = a >= 0 && a < V;
  st.z_a = has_a ? Storage<TIn>::widen(row[a]) : 0.f;
  st.member = has_a && st.z_a >= st.tau;
  st.e_a = st.member ? ex2((st.z_a - st.m) * kLog2e) : 0.f;

  // ---- sweep 2: only chunks that can hold a safe token
  const int va = has_a ? a / kPerVec : -1;
  SumCount sc = {0.f, 0};
  hot = build_hot_list(chunk_max, n_steps, st.tau, hot_smem);
  if (hot.fits()) {
    const int wbase = tid & ~31;
    for (int q = tid & 31; q < hot.count; q += 32) {
      const uint32_t e = hot.slots[q];
      const int vb = (int)(e >> 5) * per_sweep, owner = wbase + (int)(e & 31);
      Chunk<TIn, kUnroll> c;
      c.load(row, V, n_full, vb, owner);
      chunk_masked_sum<TIn, kUnroll>(c, vb, owner, a, va, st.tau, st.m, sc);
    }
  } else {
    for (int i = 0; i < n_steps; ++i) {
      if (chunk_max[i * blockDim.x + tid] >= st.tau) {
        Chunk<TIn, kUnroll> c;
        c.load(row, V, n_full, i * per_sweep, tid);
        chunk_masked_sum<TIn, kUnroll>(c, i * per_sweep, tid, a, va, st.tau, st.m, sc);
      }
    }
  }
  const SumCount tot = block_reduce_sumcount(sc, scratch);
  st.s_x = tot.s;
  st.n = tot.n;

  // ---- optional packed membership mask (diagnostic output, plain loads)
  if (mask_row) {
    const int n_words = (V + 31) / 32;
    for (int w = tid; w < n_words; w += blockDim.x) {
      uint32_t bits = 0;
      for (int b = 0; b < 32; ++b) {
        const long long k = (long long)w * 32 + b;
        if (k < V && Storage<TIn>::widen(row[k]) >= st.tau) bits |= 1u << b;
      }
      mask_row[w] = bits;
    }
  }
  return st;
}

// Gradient entries of one chunk (Prop. 5.4, set fixed), stored to the row.
template <typename TIn, typename TGrad, int kUnroll>
__device__ __forceinline__ void chunk_grad(const Chunk<TIn, kUnroll> &c, TGrad *grow, int V,
                                           int n_full, int n_vec, int vb, int tid, int a, int va,
                                           float tau, float m, float coef, float g_a) {
  constexpr int kPerVec = Storage<TIn>::kPerVec;
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    const int v = vb + u * (int)blockDim.x + tid;
    if (v >= n_vec) continue;
    float x[kPerVec], out[kPerVec];
    c.get(u, x);
    const int ja = v == va ? a - va * kPerVec : -1;
#pragma unroll
    for (int j = 0; j < kPerVec; ++j) {
      out[j] = x[j] >= tau ? coef * ex2((x[j] - m) * kLog2e) : 0.f;
      if (j == ja) out[j] = g_a;
    }
    if (v < n_full) {
      store_grads<TGrad, kPerVec>(grow + (size_t)v * kPerVec, out);
    } else {
#pragma unroll
      for (int j = 0; j < kPerVec; ++j) {
        const long long k = (long long)v * kPerVec + j;
        if (k < V) grow[k] = Storage<TGrad>::narrow(out[j]);
      }
    }
  }
}

// Sweep 3: gradient of g * ln pi^mp(a) over the row.  Chunks without a safe
// token are written as zeros without being read.
template <typename TIn, typename TGrad, int kUnroll>
__device__ __forceinline__ void row_grad(const TIn *row, TGrad *grow, int V, int a,
                                         const SideStats &st, float g, const float *chunk_max,
                                         const HotList &hot) {
  constexpr int kPerVec = Storage<TIn>::kPerVec;
  const int n_full = V / kPerVec;
  const int n_vec = (V + kPerVec - 1) / kPerVec;
  const int per_sweep = kUnroll * (int)blockDim.x;
  const int n_steps = (n_vec + per_sweep - 1) / per_sweep;
  const int tid = threadIdx.x;
  const float s_safe = st.s_x + st.e_a;
  // a pruned or missing sampled token has weight zero: the row is all zeros
  const bool live = st.member;
  const float coef = live ? -g / s_safe : 0.f;
  const float g_a = live ? g * (st.s_x / s_safe) : 0.f;
  const int va = live ? a / kPerVec : -1;
  const bool listed = live && hot.fits();
  const float tau = live ? st.tau : -kNegInf;  // +inf: nothing passes

  for (int i = 0; i < n_steps; ++i) {
    const int vb = i * per_sweep;
    if (chunk_max[i * blockDim.x + tid] >= tau) {
      if (!listed) {
        Chunk<TIn, kUnroll> c;
        c.load(row, V, n_full, vb, tid);
        chunk_grad<TIn, TGrad, kUnroll>(c, grow, V, n_full, n_vec, vb, tid, a, va, tau, st.m, coef,
                                        g_a);
      }
      continue;
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int v = vb + u * (int)blockDim.x + tid;
      if (v < n_full) {
        store_zeros<TGrad, kPerVec>(grow + (size_t)v * kPerVec);
      } else if (v < n_vec) {
        for (int j = 0; j < kPerVec; ++j) {
          const long long k = (long long)v * kPerVec + j;
          if (k < V) grow[k] = Storage<TGrad>::narrow(0.f);
        }
      }
    }
  }
  if (listed) {
    const int wbase = tid & ~31;
    for (int q = tid & 31; q < hot.count; q += 32) {
      const uint32_t e = hot.slots[q];
      const int vb = (int)(e >> 5) * per_sweep, owner = wbase + (int)(e & 31);
      Chunk<TIn, kUnroll> c;
      c.load(row, V, n_full, vb, owner);
      chunk_grad<TIn, TGrad, kUnroll>(c, grow, V, n_full, n_vec, vb, owner, a, va, tau, st.m, coef,
                                      g_a);
    }
  }
}

template <typename TIn, typename TGrad, int kUnroll>
__global__ void __launch_bounds__(512, 2) dvp_row_kernel(const RowParams p) {
  extern __shared__ __align__(16) float smem[];
  float *scratch = smem;  // 64 floats for the block reductions
  uint32_t *hot_smem = reinterpret_cast<uint32_t *>(smem + 64);  // kHotCap per warp
  float *chunk_max = smem + 64 + (blockDim.x >> 5) * kHotCap;    // one float per (step, thread)

  const long long t = blockIdx.x;
  const long long id = p.ids ? load_id(p.ids, p.id_is_i32, t) : -1;
  const bool has_id = id >= 0, bad_id = id >= p.V;
  const int a = (has_id && !bad_id) ? (int)id : -1;
  const int V = (int)p.V;

  const TIn *trow = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
  uint32_t *mask_t = p.out_t.mask ? p.out_t.mask + t * ((p.V + 31) / 32) : nullptr;
  HotList hot;
  const SideStats st =
      row_stats<TIn, kUnroll>(trow, V, a, p.log_rho, chunk_max, scratch, hot_smem, hot, mask_t);

  if (p.grad) {
    const float g = p.upstream[t];
    row_grad<TIn, TGrad, kUnroll>(trow, reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad, V, a, st,
                                  g, chunk_max, hot);
  }

  SideStats si;
  if (p.infer) {
    __syncthreads();  // chunk_max and the hot lists are reused for the second matrix
    const TIn *irow = reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer;
    uint32_t *mask_i = p.out_i.mask ? p.out_i.mask + t * ((p.V + 31) / 32) : nullptr;
    HotList hot_i;
    si = row_stats<TIn, kUnroll>(irow, V, a, p.log_rho, chunk_max, scratch, hot_smem, hot_i, mask_i);
  }

  if (threadIdx.x == 0) {
    const float lt = finish_side(p.out_t, t, st, has_id, bad_id);
    uint8_t flags = (uint8_t)((st.member ? DVP_FLAG_IN_TRAIN : 0) | (has_id ? 0 : DVP_FLAG_NO_ID) |
                              (bad_id ? DVP_FLAG_BAD_ID : 0));
    if (p.infer) {
      const float li = finish_side(p.out_i, t, si, has_id, bad_id);
      if (si.member) flags |= DVP_FLAG_IN_INFER;
      if (p.log_ratio)
        p.log_ratio[t] = (has_id && !bad_id) ? log_ratio_of(st.member, si.member, lt, li)
                                             : __int_as_float(0x7fc00000);
    }
    if (p.flags) p.flags[t] = flags;
  }
}

// ---- scalar kernel: any alignment, any row length ---------------------------
// Three plain sweeps per matrix with element-wise loads; used when a row does
// not start on a 16-byte boundary or is too long for the chunk summary.

template <typename TIn>
__device__ __forceinline__ SideStats row_stats_scalar(const TIn *row, long long V, long long a,
                                                      double log_rho, float *scratch,
                                                      uint32_t *mask_row) {
  float m = kNegInf;
  for (long long k = threadIdx.x; k < V; k += blockDim.x) m = fmaxf(m, Storage<TIn>::widen(row[k]));
  MaxSum acc = {m, 0.f};
  if (m > kNegInf)
    for (long long k = threadIdx.x; k < V; k += blockDim.x)
      acc.s += ex2((Storage<TIn>::widen(row[k]) - m) * kLog2e);
  const MaxSum all = block_reduce_maxsum(acc, scratch);
  SideStats st;
  st.m = all.m;
  st.s = all.s;
  st.tau = threshold_f32(all.m, log_rho);
  const bool has_a = a >= 0 && a < V;
  st.z_a = has_a ? Storage<TIn>::widen(row[a]) : 0.f;
  st.member = has_a && st.z_a >= st.tau;
  st.e_a = st.member ? ex2((st.z_a - st.m) * kLog2e) : 0.f;
  SumCount sc = {0.f, 0};
  for (long long k = threadIdx.x; k < V; k += blockDim.x) {
    const float z = Storage<TIn>::widen(row[k]);
    if (z >= st.tau) {
      ++sc.n;
      if (k != a) sc.s += ex2((z - st.m) * kLog2e);
    }
  }
  const SumCount tot = block_reduce_sumcount(sc, scratch);
  st.s_x = tot.s;
  st.n = tot.n;
  if (mask_row) {
    const long long n_words = (V + 31) / 32;
    for (long long w = threadIdx.x; w < n_words; w += blockDim.x) {
      uint32_t bits = 0;
      for (int b = 0; b < 32; ++b) {
        const long long k = w * 32 + b;
        if (k < V && Storage<TIn>::widen(row[k]) >= st.tau) bits |= 1u << b;
      }
      mask_row[w] = bits;
    }
  }
  return st;
}

template <typename TIn, typename TGrad>
__global__ void dvp_row_kernel_scalar(const RowParams p) {
  __shared__ float scratch[64];
  const long long t = blockIdx.x;
  const long long id = p.ids ? load_id(p.ids, p.id_is_i32, t) : -1;
  const bool has_id = id >= 0, bad_id = id >= p.V;
  const long long a = (has_id && !bad_id) ? id : -1;

  const TIn *trow = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
  uint32_t *mask_t = p.out_t.mask ? p.out_t.mask + t * ((p.V + 31) / 32) : nullptr;
  const SideStats st = row_stats_scalar<TIn>(trow, p.V, a, p.log_rho, scratch, mask_t);

  if (p.grad) {
    TGrad *grow = reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad;
    const float g = p.upstream[t];
    const float s_safe = st.s_x + st.e_a;
    const bool live = st.member;
    const float coef = live ? -g / s_safe : 0.f;
    const float g_a = live ? g * (st.s_x / s_safe) : 0.f;
    for (long long k = threadIdx.x; k < p.V; k += blockDim.x) {
      const float z = Storage<TIn>::widen(trow[k]);
      float out = (live && z >= st.tau) ? coef * ex2((z - st.m) * kLog2e) : 0.f;
      if (live && k == a) out = g_a;
      grow[k] = Storage<TGrad>::narrow(out);
    }
  }

  SideStats si;
  if (p.infer) {
    const TIn *irow = reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer;
    uint32_t *mask_i = p.out_i.mask ? p.out_i.mask + t * ((p.V + 31) / 32) : nullptr;
    si = row_stats_scalar<TIn>(irow, p.V, a, p.log_rho, scratch, mask_i);
  }

  if (threadIdx.x == 0) {
    const float lt = finish_side(p.out_t, t, st, has_id, bad_id);
    uint8_t flags = (uint8_t)((st.member ? DVP_FLAG_IN_TRAIN : 0) | (has_id ? 0 : DVP_FLAG_NO_ID) |
                              (bad_id ? DVP_FLAG_BAD_ID : 0));
    if (p.infer) {
      const float li = finish_side(p.out_i, t, si, has_id, bad_id);
      if (si.member) flags |= DVP_FLAG_IN_INFER;
      if (p.log_ratio)
        p.log_ratio[t] = (has_id && !bad_id) ? log_ratio_of(st.member, si.member, lt, li)
                                             : __int_as_float(0x7fc00000);
    }
    if (p.flags) p.flags[t] = flags;
  }
}

// ---- stand-alone backward: a streaming map from saved row statistics ---------

template <typename TIn, typename TGrad, int kUnroll, bool kVector>
__global__ void dvp_backward_kernel(const BackwardParams p) {
  constexpr int kPerVec = Storage<TIn>::kPerVec;
  const long long t = blockIdx.x;
  const TIn *row = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
  TGrad *grow = reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad;
  const long long id = load_id(p.ids, p.id_is_i32, t);
  const bool live = (p.flags[t] & DVP_FLAG_IN_TRAIN) && id >= 0 && id < p.V;
  const long long a = live ? id : -1;
  const float g = p.upstream[t], m = p.max_t[t];
  const float tau = live ? threshold_f32(m, p.log_rho) : -kNegInf;
  // e^{z - lse_safe} = e^{z - m} e^{m - lse_safe}; the second factor is 1 / s_safe
  const float coef = live ? -g * ex2((m - p.lse_safe_t[t]) * kLog2e) : 0.f;
  float g_a = 0.f;
  if (live) {
    const float comp = p.comp_mp_t ? p.comp_mp_t[t]
                                   : -expm1f(Storage<TIn>::widen(row[a]) - p.lse_safe_t[t]);
    g_a = g * comp;
  }
  if constexpr (kVector) {
    const int V = (int)p.V;
    const int n_full = V / kPerVec;
    const int n_vec = (V + kPerVec - 1) / kPerVec;
    const int per_sweep = kUnroll * (int)blockDim.x;
    const int va = live ? (int)(a / kPerVec) : -1;
    for (int vb = 0; vb < n_vec; vb += per_sweep) {
      Chunk<TIn, kUnroll> c;
      c.load(row, V, n_full, vb, threadIdx.x);
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int v = vb + u * (int)blockDim.x + threadIdx.x;
        if (v >= n_vec) continue;
        float x[kPerVec], out[kPerVec];
        c.get(u, x);
        const int ja = v == va ? (int)a - va * kPerVec : -1;
#pragma unroll
        for (int j = 0; j < kPerVec; ++j) {
          out[j] = x[j] >= tau ? coef * ex2((x[j] - m) * kLog2e) : 0.f;
          if (j == ja) out[j] = g_a;
        }
        if (v < n_full) {
          store_grads<TGrad, kPerVec>(grow + (size_t)v * kPerVec, out);
        } else {
#pragma unroll
          for (int j = 0; j < kPerVec; ++j)
            if ((long long)v * kPerVec + j < V) grow[(long long)v * kPerVec + j] = Storage<TGrad>::narrow(out[j]);
        }
      }
    }
  } else {
    for (long long k = threadIdx.x; k < p.V; k += blockDim.x) {
      const float z = Storage<TIn>::widen(row[k]);
      float out = z >= tau ? coef * ex2((z - m) * kLog2e) : 0.f;
      if (k == a) out = g_a;
      grow[k] = Storage<TGrad>::narrow(out);
    }
  }
}

// ---- host-side launchers ------------------------------------------------------

static bool aligned16(const void *base, long long ld, size_t elem) {
  return base == nullptr || (((uintptr_t)base % 16 == 0) && ((ld * (long long)elem) % 16 == 0));
}

template <typename TIn, typename TGrad, int kUnroll>
static cudaError_t launch_rows_vec(const RowParams &p, int threads, size_t smem, cudaStream_t s) {
  auto k = dvp_row_kernel<TIn, TGrad, kUnroll>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  k<<<(unsigned)p.T, threads, smem, s>>>(p);
  return cudaGetLastError();
}

template <typename TIn, typename TGrad>
static cudaError_t launch_rows(const RowParams &p, uint32_t hint, cudaStream_t s) {
  constexpr int kPerVec = Storage<TIn>::kPerVec;
  int threads = hint & 0xffff, unroll = (hint >> 16) & 0xff;
  if (threads == 0) threads = 256;
  if (unroll == 0) unroll = 4;
  const bool vec_ok = aligned16(p.train, p.ld_train, sizeof(TIn)) &&
                      aligned16(p.infer, p.ld_infer, sizeof(TIn)) &&
                      aligned16(p.grad, p.ld_grad, sizeof(TGrad));
  const long long n_vec = (p.V + kPerVec - 1) / kPerVec;
  // shrink the block for short rows so that threads are not idle
  while (threads > 64 && (long long)threads * unroll / 2 >= n_vec) threads /= 2;
  auto smem_for = [&](int u) {
    const long long per = (long long)u * threads;
    return (size_t)(64 + (threads / 32) * kHotCap + ((n_vec + per - 1) / per) * threads) * sizeof(float);
  };
  const size_t smem_cap = 200 * 1024;
  if (vec_ok) {
    if (unroll < 4) unroll = 4;
    while (unroll < 8 && smem_for(unroll) > 72 * 1024) unroll *= 2;
    if (smem_for(unroll) <= smem_cap) {
      if (unroll <= 4) return launch_rows_vec<TIn, TGrad, 4>(p, threads, smem_for(4), s);
      return launch_rows_vec<TIn, TGrad, 8>(p, threads, smem_for(8), s);
    }
  }
  dvp_row_kernel_scalar<TIn, TGrad><<<(unsigned)p.T, 512, 0, s>>>(p);
  return cudaGetLastError();
}

template <typename TIn>
static cudaError_t launch_rows_g(const RowParams &p, int grad_dtype, uint32_t hint, cudaStream_t s) {
  switch (grad_dtype) {
    case DVP_F32: return launch_rows<TIn, float>(p, hint, s);
    case DVP_BF16: return launch_rows<TIn, __nv_bfloat16>(p, hint, s);
    default: return launch_rows<TIn, __half>(p, hint, s);
  }
}

cudaError_t launch_row_kernels(const RowParams &p, int logits_dtype, int grad_dtype, uint32_t hint,
                               cudaStream_t s) {
  switch (logits_dtype) {
    case DVP_F32: return launch_rows_g<float>(p, grad_dtype, hint, s);
    case DVP_BF16: return launch_rows_g<__nv_bfloat16>(p, grad_dtype, hint, s);
    default: return launch_rows_g<__half>(p, grad_dtype, hint, s);
  }
}

template <typename TIn, typename TGrad>
static cudaError_t launch_bwd(const BackwardParams &p, uint32_t hint, cudaStream_t s) {
  int threads = hint & 0xffff;
  if (threads == 0) threads = 256;
  const bool vec_ok =
      aligned16(p.train, p.ld_train, sizeof(TIn)) && aligned16(p.grad, p.ld_grad, sizeof(TGrad));
  if (vec_ok)
    dvp_backward_kernel<TIn, TGrad, 4, true><<<(unsigned)p.T, threads, 0, s>>>(p);
  else
    dvp_backward_kernel<TIn, TGrad, 1, false><<<(unsigned)p.T, threads, 0, s>>>(p);
  return cudaGetLastError();
}

template <typename TIn>
static cudaError_t launch_bwd_g(const BackwardParams &p, int grad_dtype, uint32_t hint,
                                cudaStream_t s) {
  switch (grad_dtype) {
    case DVP_F32: return launch_bwd<TIn, float>(p, hint, s);
    case DVP_BF16: return launch_bwd<TIn, __nv_bfloat16>(p, hint, s);
    default: return launch_bwd<TIn, __half>(p, hint, s);
  }
}

cudaError_t launch_backward_kernel(const BackwardParams &p, int logits_dtype, int grad_dtype,
                                   uint32_t hint, cudaStream_t s) {
  switch (logits_dtype) {
    case DVP_F32: return launch_bwd_g<float>(p, grad_dtype, hint, s);
    case DVP_BF16: return launch_bwd_g<__nv_bfloat16>(p, grad_dtype, hint, s);
    default: return launch_bwd_g<__half>(p, grad_dtype, hint, s);
  }
}

}  // namespace dvp
