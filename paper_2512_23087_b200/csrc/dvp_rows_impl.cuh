// Row kernels of Dynamic Vocabulary Pruning for sm_100a.
//
// One thread block owns one token row.  The row is streamed from HBM once
// (sweep 1) in 32-byte granules, one DRAM sector per lane and load, two
// pipeline stages deep.  While it streams, every thread keeps an online
// log-sum-exp of what it has seen and leaves in shared memory an upper bound
// (bfloat16, rounded up) of the maximum of each granule it loaded.  Once the
// row maximum, hence the threshold of Def. 5.1, is known, only granules whose
// bound reaches the threshold can hold safe tokens: sweep 2 (masked sum and
// count, Def. 5.2) and sweep 3 (gradient, Prop. 5.4) revisit just those, and
// sweep 3 writes zeros for all the others without reading anything.  With a
// sparse safe set a row costs one HBM read per logit matrix and one HBM write
// of the gradient; with a dense safe set the same code degrades to three
// sweeps, still correct.
#pragma once
#include "dvp_common.cuh"

namespace dvp {

template <typename T>
struct Pair;
template <>
struct Pair<__nv_bfloat16> {
  using type = __nv_bfloat162;
};
template <>
struct Pair<__half> {
  using type = __half2;
};

// ---- a 32-byte granule of a row, kept packed as loaded ------------------------

template <typename TIn>
struct Granule {
  static constexpr int kElems = 32 / (int)sizeof(TIn);
  uint32_t w[8];

  __device__ __forceinline__ void load(const TIn *p) { ld_stream32(p, w); }

  // Granule `g` of a row of V elements; elements past V read as -inf.
  __device__ __forceinline__ void load_any(const TIn *row, int V, int n_full, int g) {
    // granules past the end of the row are legal here (they read as -inf); what the
    // bounds-checking build verifies is that the vector load below stays inside the row
    if (g < 0 || (g < n_full && !DVP_IN((long long)g * kElems + kElems - 1, V, DVP_OOB_GLOBAL))) {
      (void)DVP_IN(g, n_gran, DVP_OOB_GRANULE);
      const TIn fill = Storage<TIn>::narrow(kNegInf);
      uint32_t f = 0;
      if constexpr (sizeof(TIn) == 4) {
        f = *reinterpret_cast<const uint32_t *>(&fill);
      } else {
        const uint32_t h = *reinterpret_cast<const uint16_t *>(&fill);
        f = h | (h << 16);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) w[i] = f;
      return;
    }
    if (g < n_full) {
      load(row + (size_t)g * kElems);
    } else {
      __align__(16) TIn tmp[kElems];
#pragma unroll
      for (int j = 0; j < kElems; ++j) {
        const long long k = (long long)g * kElems + j;
        tmp[j] = k < V ? row[k] : Storage<TIn>::narrow(kNegInf);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) w[i] = reinterpret_cast<const uint32_t *>(tmp)[i];
    }
  }

  // Granule `g` of the row's n_full whole granules; any other index reads as -inf.  The row
  // kernel's sweeps use this one: the elements behind the last whole granule are not theirs (a few
  // threads take them one by one), so no sweep carries the element-wise code of a ragged granule.
  __device__ __forceinline__ void load_whole(const TIn *row, int n_full, int g) {
    if (g < 0 || g >= n_full || !DVP_IN((long long)g * kElems + kElems - 1, V, DVP_OOB_GLOBAL)) {
      if (g < 0) (void)DVP_IN(g, n_gran, DVP_OOB_GRANULE);
      const TIn fill = Storage<TIn>::narrow(kNegInf);
      uint32_t f = 0;
      if constexpr (sizeof(TIn) == 4) {
        f = *reinterpret_cast<const uint32_t *>(&fill);
      } else {
        const uint32_t h = *reinterpret_cast<const uint16_t *>(&fill);
        f = h | (h << 16);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) w[i] = f;
      return;
    }
    load(row + (size_t)g * kElems);
  }

  __device__ __forceinline__ void get(float *x) const {
    constexpr int kHalf = kElems / 2;
    Storage<TIn>::unpack(make_uint4(w[0], w[1], w[2], w[3]), x);
    Storage<TIn>::unpack(make_uint4(w[4], w[5], w[6], w[7]), x + kHalf);
  }

  __device__ __forceinline__ float max() const {
    if constexpr (sizeof(TIn) == 4) {
      float m = __uint_as_float(w[0]);
#pragma unroll
      for (int i = 1; i < 8; ++i) m = fmaxf(m, __uint_as_float(w[i]));
      return m;
    } else {
      // packed two-at-a-time maxima, then the two halves of the last pair
      using T2 = typename Pair<TIn>::type;
      T2 p[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) p[i] = *reinterpret_cast<const T2 *>(&w[i]);
#pragma unroll
      for (int s = 4; s > 0; s >>= 1)
#pragma unroll
        for (int i = 0; i < s; ++i) p[i] = __hmax2(p[i], p[i + s]);
      return fmaxf(Storage<TIn>::widen(p[0].x), Storage<TIn>::widen(p[0].y));
    }
  }
};

// Upper bound of a float as a bfloat16 bit pattern (round toward +inf).
__device__ __forceinline__ uint16_t bf16_bits_round_up(float v) {
  const uint32_t b = __float_as_uint(v);
  // positive: bump the magnitude unless the low half is zero; negative: truncate
  return (uint16_t)(((b & 0x80000000u) ? b : b + 0xffffu) >> 16);
}
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
  return __uint_as_float((uint32_t)b << 16);
}
// Largest bfloat16 that is <= v, as a float: comparing the stored upper bounds with
// it flags a superset of the granules whose bound reaches v.
__device__ __forceinline__ float bf16_round_down(float v) {
  const uint32_t b = __float_as_uint(v);
  return __uint_as_float(((b & 0x80000000u) ? b + 0xffffu : b) & 0xffff0000u);
}
// The bounds of one thread's kStage granules of a step sit side by side, so that a
// step's pair is one 32-bit word: slot i = step * kStage + u of thread tid.
template <int kStage>
__device__ __forceinline__ int bound_index(int slot, int tid) {
  return ((slot / kStage) * (int)blockDim.x + tid) * kStage + (slot % kStage);
}

template <typename TGrad, int kElems>
__device__ __forceinline__ void store_granule(TGrad *dst, const float *out) {
  constexpr int kBytes = kElems * (int)sizeof(TGrad);
  if constexpr (sizeof(TGrad) == 4) {
#pragma unroll
    for (int i = 0; i < kElems; i += 8) {
      uint32_t w[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) w[j] = __float_as_uint(out[i + j]);
      st_stream32(dst + i, w);
    }
  } else {
    uint32_t w[kElems / 2];
#pragma unroll
    for (int i = 0; i < kElems / 2; ++i) {
      TGrad lo = Storage<TGrad>::narrow(out[2 * i]), hi = Storage<TGrad>::narrow(out[2 * i + 1]);
      w[i] = (uint32_t) * reinterpret_cast<uint16_t *>(&lo) |
             ((uint32_t) * reinterpret_cast<uint16_t *>(&hi) << 16);
    }
    if constexpr (kBytes == 32) {
      uint32_t v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = w[i];
      st_stream32(dst, v);
    } else {
      static_assert(kBytes == 16, "granule of 8 floats stored as 8 halves");
      st_stream16(dst, make_uint4(w[0], w[1], w[2], w[3]));
    }
  }
}

template <typename TGrad, int kElems>
__device__ __forceinline__ void store_zero_granule(TGrad *dst) {
  constexpr int kBytes = kElems * (int)sizeof(TGrad);
  const uint32_t z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if constexpr (kBytes == 64) {
    st_stream32(dst, z);
    st_stream32(reinterpret_cast<char *>(dst) + 32, z);
  } else if constexpr (kBytes == 32) {
    st_stream32(dst, z);
  } else {
    st_stream16(dst, make_uint4(0, 0, 0, 0));
  }
}

// ---- granules that can hold a safe token ----------------------------------------
// Per warp, in the order (slot, lane): entry = ordinal of the granule among the
// warp's granules.  A warp whose hot granules do not fit (a dense safe set)
// walks all of its granules instead, which is then the efficient thing to do.
constexpr int kHotCap = 1024;  // 16-bit entries: slot * 32 + lane stays below 65536 for every row the bounds fit

struct HotList {
  uint16_t *slots;
  int count;  // granules at or above the threshold (may exceed kHotCap)
  __device__ __forceinline__ bool fits() const { return count <= kHotCap; }
};

// tau_b: the threshold rounded down to bfloat16.  Each thread first gathers the
// flags of its own slots into a register (16 steps at a time: one packed compare per
// step), then a warp prefix sum hands out list positions: the cost of the scan does
// not depend on how many granules are hot, and the order of the list is fixed.
template <int kStage>
__device__ __forceinline__ HotList build_hot_list(const uint16_t *bound, int n_steps, float tau_b,
                                                  uint16_t *hot_smem) {
  static_assert(kStage == 2, "the packed scan reads the two bounds of a step as one word");
  const int lane = threadIdx.x & 31, tid = threadIdx.x;
  HotList h;
  h.slots = hot_smem + (tid >> 5) * kHotCap;
  h.count = 0;
  const uint32_t *words = reinterpret_cast<const uint32_t *>(bound);
  const __nv_bfloat16 tb = __float2bfloat16_rz(tau_b);  // exact: tau_b is a bfloat16 value
  const __nv_bfloat162 tau2 = __halves2bfloat162(tb, tb);
  for (int step0 = 0; step0 < n_steps; step0 += 16) {
    uint32_t acc = 0;  // bit s: first granule of step step0 + s, bit 16 + s: second granule
    const int n = min(16, n_steps - step0);
    for (int s = 0; s < n; ++s) {
      const int wi = (step0 + s) * (int)blockDim.x + tid;
      const uint32_t w = DVP_IN(2 * wi + 1, n_bound, DVP_OOB_BOUND) ? words[wi] : 0u;
      const uint32_t m = __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&w), tau2);
      acc |= (m & 0x00010001u) << s;
    }
    const int cnt = __popc(acc);
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    int pos = h.count + incl - cnt;
    while (acc) {
      const int b = __ffs(acc) - 1;
      acc &= acc - 1;
      const int slot = (step0 + (b & 15)) * 2 + (b >> 4);
      if (pos < kHotCap) h.slots[pos] = (uint16_t)(slot * 32 + lane);
      ++pos;
    }
    h.count += __shfl_sync(0xffffffffu, incl, 31);
  }
  __syncwarp();
  return h;
}

// Contribution of one granule to the masked sum and the count (Def. 5.2).
template <typename TIn>
__device__ __forceinline__ void granule_masked_sum(const Granule<TIn> &gr, int g, int a, float tau,
                                                   float m, SumCount &sc) {
  constexpr int kElems = Granule<TIn>::kElems;
  float x[kElems];
  gr.get(x);
  // the sampled token is left out so that 1 - pi^mp(a) has no cancellation
  const int ja = a - g * kElems;  // in [0, kElems) only inside the owner granule
#pragma unroll
  for (int j = 0; j < kElems; ++j) {
    if (x[j] >= tau && x[j] > kNegInf) {  // the fill of a ragged last granule is never a token
      ++sc.n;
      if (j != ja) sc.s += ex2((x[j] - m) * kLog2e);
    }
  }
}

// Gradient entries of one granule (Prop. 5.4, set fixed), stored to the row.
template <typename TIn, typename TGrad>
__device__ __forceinline__ void granule_grad(const Granule<TIn> &gr, TGrad *grow, int V, int n_full,
                                             int g, int a, float tau, float m, float coef,
                                             float g_a) {
  constexpr int kElems = Granule<TIn>::kElems;
  float x[kElems], out[kElems];
  gr.get(x);
  const int ja = a - g * kElems;
#pragma unroll
  for (int j = 0; j < kElems; ++j) {
    out[j] = x[j] >= tau ? coef * ex2((x[j] - m) * kLog2e) : 0.f;
    if (j == ja) out[j] = g_a;
  }
  // a granule past the end of the row is legal here (a hot list built for a threshold of -inf
  // names them): nothing of it is stored below.  A negative index is not.
  if (g < 0) {
    (void)DVP_IN(g, n_gran, DVP_OOB_GRANULE);
    return;
  }
  if (g < n_full) {
    if (!DVP_IN((long long)g * kElems + kElems - 1, V, DVP_OOB_GLOBAL)) return;
    store_granule<TGrad, kElems>(grow + (size_t)g * kElems, out);
  } else {
#pragma unroll
    for (int j = 0; j < kElems; ++j) {
      const long long k = (long long)g * kElems + j;
      if (k < V) grow[k] = Storage<TGrad>::narrow(out[j]);
    }
  }
}

// The same for a whole granule of the row kernel's sweeps (nothing is stored for any other index).
template <typename TIn, typename TGrad>
__device__ __forceinline__ void granule_grad_whole(const Granule<TIn> &gr, TGrad *grow, int n_full, int g, int a,
                                                   float tau, float m, float coef, float g_a) {
  constexpr int kElems = Granule<TIn>::kElems;
  if (g < 0 || g >= n_full) {
    if (g < 0) (void)DVP_IN(g, n_gran, DVP_OOB_GRANULE);
    return;
  }
  float x[kElems], out[kElems];
  gr.get(x);
  const int ja = a - g * kElems;
#pragma unroll
  for (int j = 0; j < kElems; ++j) {
    out[j] = x[j] >= tau ? coef * ex2((x[j] - m) * kLog2e) : 0.f;
    if (j == ja) out[j] = g_a;
  }
  if (!DVP_IN((long long)g * kElems + kElems - 1, V, DVP_OOB_GLOBAL)) return;
  store_granule<TGrad, kElems>(grow + (size_t)g * kElems, out);
}

// One pipeline stage of sweep 1: kStage granules of this thread.
template <typename TIn, int kStage>
struct Stage {
  Granule<TIn> g[kStage];
  // every granule of the step, the elements of a ragged last granule included
  __device__ __forceinline__ void load(const TIn *row, int V, int n_full, int step) {
    const int g0 = step * kStage * (int)blockDim.x + threadIdx.x;
    if ((step + 1) * kStage * (int)blockDim.x <= n_full &&
        DVP_IN(g0 + (kStage - 1) * (int)blockDim.x, n_gran, DVP_OOB_GRANULE)) {
#pragma unroll
      for (int u = 0; u < kStage; ++u)
        g[u].load(row + (size_t)(g0 + u * (int)blockDim.x) * Granule<TIn>::kElems);
    } else {
#pragma unroll
      for (int u = 0; u < kStage; ++u) g[u].load_any(row, V, n_full, g0 + u * (int)blockDim.x);
    }
  }
  // the whole granules of the step only
  __device__ __forceinline__ void load_whole(const TIn *row, int n_full, int step) {
    const int g0 = step * kStage * (int)blockDim.x + threadIdx.x;
    if ((step + 1) * kStage * (int)blockDim.x <= n_full &&
        DVP_IN(g0 + (kStage - 1) * (int)blockDim.x, n_gran, DVP_OOB_GRANULE)) {
#pragma unroll
      for (int u = 0; u < kStage; ++u)
        g[u].load(row + (size_t)(g0 + u * (int)blockDim.x) * Granule<TIn>::kElems);
    } else {
#pragma unroll
      for (int u = 0; u < kStage; ++u) g[u].load_whole(row, n_full, g0 + u * (int)blockDim.x);
    }
  }
};

template <typename TIn, int kStage>
__device__ __forceinline__ void absorb_stage(const Stage<TIn, kStage> &st, int step, LogSum &acc,
                                             uint16_t *bound) {
  constexpr int kElems = Granule<TIn>::kElems;
  float cm = kNegInf;
#pragma unroll
  for (int u = 0; u < kStage; ++u) {
    const float gm = st.g[u].max();
    const int bi = bound_index<kStage>(step * kStage + u, threadIdx.x);
    if (DVP_IN(bi, n_bound, DVP_OOB_BOUND)) bound[bi] = bf16_bits_round_up(gm);
    cm = fmaxf(cm, gm);
  }
  if (cm > kNegInf) {
    if (cm > acc.m) {
      const float cn = cm * kLog2e;
      acc.s *= ex2(acc.c - cn);  // acc.c = -inf at the start: the factor is 0
      acc.m = cm;
      acc.c = cn;
    }
    const float neg_c = -acc.c;
    float part = 0.f;
#pragma unroll
    for (int u = 0; u < kStage; ++u) {
      float x[kElems];
      st.g[u].get(x);
#pragma unroll
      for (int j = 0; j < kElems; ++j) part += ex2(fmaf(x[j], kLog2e, neg_c));
    }
    acc.s += part;
  }
}

// ---- a row split over a thread-block cluster -----------------------------------
// With kCluster > 1 the blocks of a cluster share one row: block `rank` owns a
// contiguous part of it, partial results meet through distributed shared memory.
// Fewer rows are then in flight (one per cluster instead of one per block), so
// the granules that sweeps 2 and 3 revisit are still in L2.

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(const float *local, uint32_t rank) {
  uint32_t laddr = (uint32_t)__cvta_generic_to_shared(local), raddr;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(laddr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(raddr) : "memory");
  return v;
}

// slot: 4 floats of this block's shared memory, written once per kernel.
template <int kCluster>
__device__ __forceinline__ LogSum cluster_reduce_logsum(LogSum v, float *slot) {
  if constexpr (kCluster == 1) return v;
  if (threadIdx.x == 0) {
    slot[0] = v.m;
    slot[1] = v.c;
    slot[2] = v.s;
  }
  cluster_sync_all();
  LogSum r = {kNegInf, kNegInf, 0.f};
#pragma unroll
  for (uint32_t k = 0; k < (uint32_t)kCluster; ++k) {  // rank order: same result in every block
    LogSum o;
    o.m = ld_cluster_f32(slot + 0, k);
    o.c = ld_cluster_f32(slot + 1, k);
    o.s = ld_cluster_f32(slot + 2, k);
    r = combine(r, o);
  }
  return r;
}

template <int kCluster>
__device__ __forceinline__ SumCount cluster_reduce_sumcount(SumCount v, float *slot) {
  if constexpr (kCluster == 1) return v;
  if (threadIdx.x == 0) {
    slot[0] = v.s;
    slot[1] = __int_as_float(v.n);
  }
  cluster_sync_all();
  SumCount r = {0.f, 0};
#pragma unroll
  for (uint32_t k = 0; k < (uint32_t)kCluster; ++k) {
    r.s += ld_cluster_f32(slot + 0, k);
    r.n += __float_as_int(ld_cluster_f32(slot + 1, k));
  }
  return r;
}

// Sweep 1 over (a part of) a row: block-wide log-sum-exp state; granule bounds
// are left in shared memory.
template <typename TIn, int kStage>
__device__ __forceinline__ LogSum row_sweep1(const TIn *row, int V, uint16_t *bound, float *scratch) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int n_full = V / kElems;  // the sweeps take whole granules; see row_tail
  const int per_step = kStage * (int)blockDim.x;
  const int n_steps = (n_full + per_step - 1) / per_step;
  LogSum acc = {kNegInf, kNegInf, 0.f};
  if (n_steps > 0) {  // two stages in flight
    Stage<TIn, kStage> s0, s1;
    s0.load_whole(row, n_full, 0);
    int step = 0;
    for (; step + 1 < n_steps; step += 2) {
      s1.load_whole(row, n_full, step + 1);
      absorb_stage<TIn, kStage>(s0, step, acc, bound);
      if (step + 2 < n_steps) s0.load_whole(row, n_full, step + 2);
      absorb_stage<TIn, kStage>(s1, step + 1, acc, bound);
    }
    if (step < n_steps) absorb_stage<TIn, kStage>(s0, step, acc, bound);
  }
  // the elements behind the last whole granule, one per thread
  const int k_tail = n_full * kElems + (int)threadIdx.x;
  if (k_tail < V) {
    const float x = Storage<TIn>::widen(row[k_tail]);
    if (x > kNegInf) {
      if (x > acc.m) {
        const float cn = x * kLog2e;
        acc.s *= ex2(acc.c - cn);
        acc.m = x;
        acc.c = cn;
      }
      acc.s += ex2(fmaf(x, kLog2e, -acc.c));
    }
  }
  return block_reduce_logsum(acc, scratch);
}

// Sweep 2 over (a part of) a row: masked sum without the sampled token and count,
// block-wide.  `a` is relative to `row` (outside [0, V): not in this part).
template <typename TIn, int kStage>
__device__ __forceinline__ SumCount row_sweep2(const TIn *row, int V, int a, float tau, float m,
                                               const uint16_t *bound, float *scratch,
                                               uint16_t *hot_smem, HotList &hot) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int n_full = V / kElems;
  const int per_step = kStage * (int)blockDim.x;
  const int n_slots = ((n_full + per_step - 1) / per_step) * kStage;  // whole granules per thread
  const int tid = threadIdx.x;
  SumCount sc = {0.f, 0};
  {  // the elements behind the last whole granule, one per thread
    const int k_tail = n_full * kElems + tid;
    if (k_tail < V) {
      const float x = Storage<TIn>::widen(row[k_tail]);
      if (x >= tau && x > kNegInf) {
        ++sc.n;
        if (k_tail != a) sc.s += ex2((x - m) * kLog2e);
      }
    }
  }
  const float tau_b = bf16_round_down(tau);
  hot = build_hot_list<kStage>(bound, n_slots / kStage, tau_b, hot_smem);
  if (hot.fits()) {
    const int wbase = tid & ~31, lane = tid & 31;
    for (int q = lane; q < hot.count; q += 64) {
      if (!DVP_IN(q, n_hot, DVP_OOB_HOT)) break;
      const uint32_t e0 = hot.slots[q];
      const bool two = q + 32 < hot.count && DVP_IN(q + 32, n_hot, DVP_OOB_HOT);
      const uint32_t e1 = two ? hot.slots[q + 32] : e0;
      const int g0 = (int)(e0 >> 5) * (int)blockDim.x + wbase + (int)(e0 & 31);
      const int g1 = (int)(e1 >> 5) * (int)blockDim.x + wbase + (int)(e1 & 31);
      Granule<TIn> a0, a1;
      a0.load_whole(row, n_full, g0);
      if (two) a1.load_whole(row, n_full, g1);
      granule_masked_sum<TIn>(a0, g0, a, tau, m, sc);
      if (two) granule_masked_sum<TIn>(a1, g1, a, tau, m, sc);
    }
  } else {
    // a dense safe set: all of the thread's granules, a step's two at a time (both loads before either is used)
    static_assert(kStage == 2, "a step's two bounds are neighbours");
    for (int i = 0; i < n_slots; i += 2) {
      if (!DVP_IN(bound_index<kStage>(i + 1, tid), n_bound, DVP_OOB_BOUND)) break;
      const bool hot0 = bf16_bits_to_float(bound[bound_index<kStage>(i, tid)]) >= tau_b;
      const bool hot1 = bf16_bits_to_float(bound[bound_index<kStage>(i + 1, tid)]) >= tau_b;
      const int g0 = i * (int)blockDim.x + tid, g1 = g0 + (int)blockDim.x;
      Granule<TIn> a0, a1;
      if (hot0) a0.load_whole(row, n_full, g0);
      if (hot1) a1.load_whole(row, n_full, g1);
      if (hot0) granule_masked_sum<TIn>(a0, g0, a, tau, m, sc);
      if (hot1) granule_masked_sum<TIn>(a1, g1, a, tau, m, sc);
    }
  }
  return block_reduce_sumcount(sc, scratch);
}

// Statistics of one side of one row.  `row` is the whole row (V elements); this
// block sweeps the part [off, off + v_part) of it.
template <typename TIn, int kStage, int kCluster>
__device__ __forceinline__ SideStats row_stats(const TIn *row, int V, int off, int v_part, int a,
                                               double log_rho, int mode, float mask_value,
                                               uint16_t *bound, float *scratch, float *cl_slots,
                                               uint16_t *hot_smem, HotList &hot) {
  const LogSum part = row_sweep1<TIn, kStage>(row + off, v_part, bound, scratch);
  const LogSum all = cluster_reduce_logsum<kCluster>(part, cl_slots);

  SideStats st;
  st.m = all.m;
  st.lse = lse_from_logsum(all);
  st.sum_c = (double)all.c;
  st.sum_s = all.s;
  st.tau = threshold_of<TIn>(all.m, log_rho, mode);
  const bool has_a = a >= 0 && a < V;
  st.z_a = has_a ? Storage<TIn>::widen(row[a]) : 0.f;
  st.member = has_a && st.z_a >= st.tau;
  st.e_a = st.member ? ex2((st.z_a - st.m) * kLog2e) : 0.f;

  const int a_part = (has_a && a >= off && a < off + v_part) ? a - off : -1;
  const SumCount sc = row_sweep2<TIn, kStage>(row + off, v_part, a_part, st.tau, st.m, bound,
                                              scratch, hot_smem, hot);
  const SumCount tot = cluster_reduce_sumcount<kCluster>(sc, cl_slots + 4);
  st.s_x = tot.s;
  st.n = tot.n;
  set_mask_mass(st, V, mode, Storage<TIn>::widen(Storage<TIn>::narrow(mask_value)), has_a);

  return st;
}

// The optional packed membership mask of a row (a diagnostic output): plain loads, one 32-bit word
// per thread and step.  Called at the end of the kernel, so that its code lies behind the sweeps'.
template <typename TIn>
__device__ __forceinline__ void write_mask_row(const TIn *row, int V, float tau, uint32_t *mask_row) {
  const int n_words = (V + 31) / 32;
  for (int w = threadIdx.x; w < n_words; w += blockDim.x) {
    uint32_t bits = 0;
    for (int b = 0; b < 32; ++b) {
      const long long k = (long long)w * 32 + b;
      if (k < V && Storage<TIn>::widen(row[k]) >= tau) bits |= 1u << b;
    }
    mask_row[w] = bits;
  }
}

// Sweep 3: gradient of g * ln pi^mp(a) over the row.  Granules without a safe
// token are written as zeros without being read.
template <typename TIn, typename TGrad, int kStage>
__device__ __forceinline__ void row_grad(const TIn *row, TGrad *grow, int V, int a,
                                         const SideStats &st, float g, const uint16_t *bound,
                                         const HotList &hot) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int n_full = V / kElems;
  const int per_step = kStage * (int)blockDim.x;
  const int n_slots = ((n_full + per_step - 1) / per_step) * kStage;
  const int tid = threadIdx.x;
  const float s_tot = st.s_x + st.e_a + st.s_mask;
  // a missing sampled token, or a pruned one under the -inf semantics, has weight zero:
  // the row is all zeros
  const bool live = st.live;
  const float coef = live ? -g / s_tot : 0.f;
  const float g_a = st.member ? g * ((st.s_x + st.s_mask) / s_tot) : 0.f;
  const int a_live = (live && st.member) ? a : -1;
  const bool listed = live && hot.fits();
  const float tau = live ? st.tau : -kNegInf;  // +inf: nothing passes
  const float tau_b = live ? bf16_round_down(st.tau) : -kNegInf;

  {  // the elements behind the last whole granule, one per thread
    const int k_tail = n_full * kElems + tid;
    if (k_tail < V) {
      const float x = Storage<TIn>::widen(row[k_tail]);
      float out = x >= tau ? coef * ex2((x - st.m) * kLog2e) : 0.f;
      if (k_tail == a_live) out = g_a;
      grow[k_tail] = Storage<TGrad>::narrow(out);
    }
  }
  for (int i = 0; i < n_slots; ++i) {
    const int gi = i * (int)blockDim.x + tid;
    if (gi >= n_full) break;
    if (!DVP_IN(bound_index<kStage>(i, tid), n_bound, DVP_OOB_BOUND)) break;
    if (bf16_bits_to_float(bound[bound_index<kStage>(i, tid)]) >= tau_b) {
      // a granule that can hold safe tokens: written below
    } else if (DVP_IN((long long)gi * kElems + kElems - 1, V, DVP_OOB_GLOBAL)) {
      store_zero_granule<TGrad, kElems>(grow + (size_t)gi * kElems);
    }
  }
  if (live && !listed) {
    // a dense safe set: all of the thread's hot granules, a step's two at a time (both loads before either is used)
    static_assert(kStage == 2, "a step's two bounds are neighbours");
    for (int i = 0; i < n_slots; i += 2) {
      if (!DVP_IN(bound_index<kStage>(i + 1, tid), n_bound, DVP_OOB_BOUND)) break;
      const int g0 = i * (int)blockDim.x + tid, g1 = g0 + (int)blockDim.x;
      const bool hot0 = g0 < n_full && bf16_bits_to_float(bound[bound_index<kStage>(i, tid)]) >= tau_b;
      const bool hot1 = g1 < n_full && bf16_bits_to_float(bound[bound_index<kStage>(i + 1, tid)]) >= tau_b;
      Granule<TIn> a0, a1;
      if (hot0) a0.load_whole(row, n_full, g0);
      if (hot1) a1.load_whole(row, n_full, g1);
      if (hot0) granule_grad_whole<TIn, TGrad>(a0, grow, n_full, g0, a_live, tau, st.m, coef, g_a);
      if (hot1) granule_grad_whole<TIn, TGrad>(a1, grow, n_full, g1, a_live, tau, st.m, coef, g_a);
    }
  }
  if (listed) {
    const int wbase = tid & ~31, lane = tid & 31;
    for (int q = lane; q < hot.count; q += 64) {
      if (!DVP_IN(q, n_hot, DVP_OOB_HOT)) break;
      const uint32_t e0 = hot.slots[q];
      const bool two = q + 32 < hot.count && DVP_IN(q + 32, n_hot, DVP_OOB_HOT);
      const uint32_t e1 = two ? hot.slots[q + 32] : e0;
      const int g0 = (int)(e0 >> 5) * (int)blockDim.x + wbase + (int)(e0 & 31);
      const int g1 = (int)(e1 >> 5) * (int)blockDim.x + wbase + (int)(e1 & 31);
      Granule<TIn> a0, a1;
      a0.load_whole(row, n_full, g0);
      if (two) a1.load_whole(row, n_full, g1);
      granule_grad_whole<TIn, TGrad>(a0, grow, n_full, g0, a_live, tau, st.m, coef, g_a);
      if (two) granule_grad_whole<TIn, TGrad>(a1, grow, n_full, g1, a_live, tau, st.m, coef, g_a);
    }
  }
}

// Shared-memory layout of the row kernel, in 4-byte words: 96 for the block
// reductions, 16 for the cluster exchange, then the hot lists, then the bounds.
__host__ __device__ inline int smem_words_fixed(int threads) {
  return 96 + 16 + (threads / 32) * kHotCap / 2;
}

// kThreads / kBlocks: the launch bounds (largest block, blocks per SM) that set
// the register budget of this instantiation.  kCluster blocks share one row.
// kWeighted: the upstream gradient is multiplied by the token's importance weight, which
// needs the inference side's statistics before sweep 3 of the training row: that
// instantiation sweeps the inference row first.
template <typename TIn, typename TGrad, int kStage, int kThreads, int kBlocks, int kCluster, bool kWeighted>
__global__ void __launch_bounds__(kThreads, kBlocks) dvp_row_kernel(const RowParams p) {
  extern __shared__ __align__(16) float smem[];
  float *scratch = smem;        // 96 floats for the block reductions
  float *cl_slots = smem + 96;  // 4 exchanges x 4 floats, each written once
  uint16_t *hot_smem = reinterpret_cast<uint16_t *>(smem + 112);  // kHotCap per warp
  uint16_t *bound = reinterpret_cast<uint16_t *>(smem + smem_words_fixed(blockDim.x));

  constexpr int kElems = Granule<TIn>::kElems;
  DVP_BOUNDS_BEGIN(p.bounds_status);
  const long long t = blockIdx.x / kCluster;
  const int rank = kCluster > 1 ? (int)cluster_rank() : 0;
  const long long id = p.ids ? load_id(p.ids, p.id_is_i32, t) : -1;
  const bool has_id = id >= 0, bad_id = id >= p.V;
  const int a = (has_id && !bad_id) ? (int)id : -1;
  const int V = (int)p.V;
  // this block's part of the row, in whole granules
  const int n_gran = (V + kElems - 1) / kElems;
  const int per_rank = (n_gran + kCluster - 1) / kCluster;
  const int off = min(rank * per_rank, n_gran) * kElems;
  const int v_part = max(0, min(V - off, per_rank * kElems));
#ifdef DVP_DEBUG_BOUNDS
  {  // extents of this block's part of the row and of its tables
    const int part_gran = (v_part + kElems - 1) / kElems, per_step = kStage * (int)blockDim.x;
    DVP_BOUNDS_SET(n_gran, part_gran);
    DVP_BOUNDS_SET(V, v_part);
    DVP_BOUNDS_SET(n_bound, (long long)((part_gran + per_step - 1) / per_step) * per_step);
    DVP_BOUNDS_SET(n_hot, kHotCap);  // entries of one warp's hot list
    DVP_BOUNDS_SYNC();
  }
#endif

  const TIn *trow = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
  uint32_t *mask_t = p.out_t.mask ? p.out_t.mask + t * ((p.V + 31) / 32) : nullptr;
  HotList hot;
  SideStats st, si;
  if (kWeighted && p.infer) {  // otherwise an earlier launch left the inference side's results
    const TIn *irow = reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer;
    HotList hot_i;
    si = row_stats<TIn, kStage, kCluster>(irow, V, off, v_part, a, p.log_rho, p.mode, p.mask_value, bound,
                                          scratch, cl_slots + 8, hot_smem, hot_i);
    __syncthreads();  // the bounds and the hot lists are reused for the second matrix
  }
  st = row_stats<TIn, kStage, kCluster>(trow, V, off, v_part, a, p.log_rho, p.mode, p.mask_value, bound,
                                        scratch, cl_slots, hot_smem, hot);

  if (p.grad) {
    float g = p.upstream[t];
    if constexpr (kWeighted) {
      const float w = p.infer ? row_weight(p, st, si, a >= 0) : row_weight_given(p, st, t, a >= 0);
      if (w == w) g *= w;
      if (p.weight_out && threadIdx.x == 0 && rank == 0) p.weight_out[t] = w;
    }
    const int a_part = (a >= off && a < off + v_part) ? a - off : -1;
    row_grad<TIn, TGrad, kStage>(trow + off, reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad + off,
                                 v_part, a_part, st, g, bound, hot);
  }

  if constexpr (!kWeighted) {
    if (p.infer) {
      __syncthreads();  // the bounds and the hot lists are reused for the second matrix
      const TIn *irow = reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer;
      HotList hot_i;
      si = row_stats<TIn, kStage, kCluster>(irow, V, off, v_part, a, p.log_rho, p.mode, p.mask_value,
                                            bound, scratch, cl_slots + 8, hot_smem, hot_i);
    }
  }

  if (threadIdx.x == 0 && rank == 0) {
    const float lt = finish_side(p.out_t, t, st, has_id, bad_id);
    uint8_t flags = (uint8_t)((st.member ? DVP_FLAG_IN_TRAIN : 0) | (has_id ? 0 : DVP_FLAG_NO_ID) |
                              (bad_id ? DVP_FLAG_BAD_ID : 0));
    if (p.infer) {
      const float li = finish_side(p.out_i, t, si, has_id, bad_id);
      if (si.member) flags |= DVP_FLAG_IN_INFER;
      if (p.log_ratio)
        p.log_ratio[t] = !(has_id && !bad_id)              ? __int_as_float(0x7fc00000)
                         : (p.mode & DVP_MODE_FINITE_MASK) ? lt - li
                                                           : log_ratio_of(st.member, si.member, lt, li);
    }
    if (p.flags) p.flags[t] = flags;
  }
  if (off == 0) {  // the first block of a row's cluster writes the row's masks
    if (mask_t) write_mask_row<TIn>(trow, V, st.tau, mask_t);
    if (p.infer && p.out_i.mask)
      write_mask_row<TIn>(reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer, V, si.tau,
                          p.out_i.mask + t * ((p.V + 31) / 32));
  }
  // no block may leave while another one can still read its exchange slots
  if constexpr (kCluster > 1) cluster_sync_all();
}

// ---- scalar kernel: any alignment, any row length ---------------------------
// Three plain sweeps per matrix with element-wise loads; used when a row does
// not start on a 32-byte boundary or is too long for the granule bounds.

template <typename TIn>
__device__ __forceinline__ SideStats row_stats_scalar(const TIn *row, long long V, long long a,
                                                      double log_rho, int mode, float mask_value,
                                                      float *scratch, uint32_t *mask_row) {
  float m = kNegInf;
  for (long long k = threadIdx.x; k < V; k += blockDim.x) m = fmaxf(m, Storage<TIn>::widen(row[k]));
  MaxSum acc = {m, 0.f};
  if (m > kNegInf)
    for (long long k = threadIdx.x; k < V; k += blockDim.x)
      acc.s += ex2((Storage<TIn>::widen(row[k]) - m) * kLog2e);
  const MaxSum all = block_reduce_maxsum(acc, scratch);
  SideStats st;
  st.m = all.m;
  st.lse = (double)all.m + (double)logf(all.s);
  st.sum_c = (double)all.m * (double)kLog2e;
  st.sum_s = all.s;
  st.tau = threshold_of<TIn>(all.m, log_rho, mode);
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
  set_mask_mass(st, V, mode, Storage<TIn>::widen(Storage<TIn>::narrow(mask_value)), has_a);
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
  const TIn *irow = p.infer ? reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer : nullptr;
  uint32_t *mask_t = p.out_t.mask ? p.out_t.mask + t * ((p.V + 31) / 32) : nullptr;
  uint32_t *mask_i = p.out_i.mask ? p.out_i.mask + t * ((p.V + 31) / 32) : nullptr;
  const SideStats st =
      row_stats_scalar<TIn>(trow, p.V, a, p.log_rho, p.mode, p.mask_value, scratch, mask_t);
  SideStats si;
  if (irow) si = row_stats_scalar<TIn>(irow, p.V, a, p.log_rho, p.mode, p.mask_value, scratch, mask_i);
  float w = 1.f;
  if (p.weight_kind != DVP_WEIGHT_NONE)
    w = irow ? row_weight(p, st, si, a >= 0) : row_weight_given(p, st, t, a >= 0);
  if (p.weight_out && threadIdx.x == 0) p.weight_out[t] = w;

  if (p.grad) {
    TGrad *grow = reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad;
    float g = p.upstream[t];
    if (w == w) g *= w;
    const float s_tot = st.s_x + st.e_a + st.s_mask;
    const bool live = st.live;
    const float coef = live ? -g / s_tot : 0.f;
    const float g_a = st.member ? g * ((st.s_x + st.s_mask) / s_tot) : 0.f;
    for (long long k = threadIdx.x; k < p.V; k += blockDim.x) {
      const float z = Storage<TIn>::widen(trow[k]);
      float out = (live && z >= st.tau) ? coef * ex2((z - st.m) * kLog2e) : 0.f;
      if (live && st.member && k == a) out = g_a;
      grow[k] = Storage<TGrad>::narrow(out);
    }
  }

  if (threadIdx.x == 0) {
    const float lt = finish_side(p.out_t, t, st, has_id, bad_id);
    uint8_t flags = (uint8_t)((st.member ? DVP_FLAG_IN_TRAIN : 0) | (has_id ? 0 : DVP_FLAG_NO_ID) |
                              (bad_id ? DVP_FLAG_BAD_ID : 0));
    if (p.infer) {
      const float li = finish_side(p.out_i, t, si, has_id, bad_id);
      if (si.member) flags |= DVP_FLAG_IN_INFER;
      if (p.log_ratio)
        p.log_ratio[t] = !(has_id && !bad_id)              ? __int_as_float(0x7fc00000)
                         : (p.mode & DVP_MODE_FINITE_MASK) ? lt - li
                                                           : log_ratio_of(st.member, si.member, lt, li);
    }
    if (p.flags) p.flags[t] = flags;
  }
}

// ---- stand-alone backward: a streaming map from saved row statistics ---------

template <typename TIn, typename TGrad, int kStage, bool kVector>
__global__ void dvp_backward_kernel(const BackwardParams p) {
  const long long t = blockIdx.x;
  DVP_BOUNDS_BEGIN(p.bounds_status);
  DVP_BOUNDS_SET(n_gran, (p.V + Granule<TIn>::kElems - 1) / Granule<TIn>::kElems);
  DVP_BOUNDS_SET(V, p.V);
  DVP_BOUNDS_SYNC();
  const TIn *row = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
  TGrad *grow = reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad;
  const long long id = load_id(p.ids, p.id_is_i32, t);
  const bool member = (p.flags[t] & DVP_FLAG_IN_TRAIN) && id >= 0 && id < p.V;
  // with a finite mask value a pruned sampled token still has a gradient on the kept positions
  const bool live = member || ((p.mode & DVP_MODE_FINITE_MASK) && id >= 0 && id < p.V);
  const long long a = member ? id : -1;
  const float g = p.upstream[t], m = p.max_t[t];
  const float tau = live ? threshold_of<TIn>(m, p.log_rho, p.mode) : -kNegInf;
  // e^{z - lse_safe} = e^{z - m} e^{m - lse_safe}; the second factor is 1 / s_safe
  const float coef = live ? -g * ex2((m - p.lse_safe_t[t]) * kLog2e) : 0.f;
  float g_a = 0.f;
  if (member) {
    const float comp = p.comp_mp_t ? p.comp_mp_t[t]
                                   : -expm1f(Storage<TIn>::widen(row[a]) - p.lse_safe_t[t]);
    g_a = g * comp;
  }
  if constexpr (kVector) {
    constexpr int kElems = Granule<TIn>::kElems;
    const int V = (int)p.V;
    const int n_full = V / kElems;
    const int n_gran = (V + kElems - 1) / kElems;
    const int per_step = kStage * (int)blockDim.x;
    for (int gb = 0; gb < n_gran; gb += per_step) {
      Granule<TIn> gr[kStage];
#pragma unroll
      for (int u = 0; u < kStage; ++u) {
        const int gi = gb + u * (int)blockDim.x + threadIdx.x;
        if (gi < n_gran) gr[u].load_any(row, V, n_full, gi);
      }
#pragma unroll
      for (int u = 0; u < kStage; ++u) {
        const int gi = gb + u * (int)blockDim.x + threadIdx.x;
        if (gi < n_gran)
          granule_grad<TIn, TGrad>(gr[u], grow, V, n_full, gi, (int)a, tau, m, coef, g_a);
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


}  // namespace dvp
#include "dvp_rows_resident.cuh"
#include "dvp_rows_store.cuh"
namespace dvp {

// ---- host-side launchers, instantiated once per logits type -------------------

static inline bool aligned32(const void *base, long long ld, size_t elem) {
  return base == nullptr || (((uintptr_t)base % 32 == 0) && ((ld * (long long)elem) % 32 == 0));
}

template <typename TIn, typename TGrad, int kStage, int kThreads, int kBlocks, int kCluster, bool kWeighted = false>
static cudaError_t launch_rows_vec(const RowParams &p, int threads, size_t smem, cudaStream_t s) {
  auto k = dvp_row_kernel<TIn, TGrad, kStage, kThreads, kBlocks, kCluster, kWeighted>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  if constexpr (kCluster == 1) {
    k<<<(unsigned)p.T, threads, smem, s>>>(p);
    return cudaGetLastError();
  } else {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.T * kCluster), 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k, p);
  }
}

// Shared memory one SM can give to `blocks` resident blocks (228 KB per SM, 1 KB of it
// reserved per block), and the most one block may ask for.
static inline size_t smem_per_block(int blocks) {
  const size_t share = (size_t)228 * 1024 / blocks - 1024;
  return share < (size_t)227 * 1024 ? share : (size_t)227 * 1024;
}

// The kernel that keeps the candidates of the safe set on chip (2-byte logits).
template <typename TIn, typename TGrad, int kThreads, int kBlocks, bool kWeighted>
static cudaError_t launch_rows_cs(const RowParams &p, int threads, int n_steps, cudaStream_t s) {
  auto k = cs::dvp_row_kernel_cs<TIn, TGrad, kThreads, kBlocks, kWeighted>;
  if (n_steps > 64) return cudaErrorNotSupported;  // positions are 16 bits
  // as many list entries per warp as the SM's shared memory allows with kBlocks blocks
  // resident, at most every element the warp sees
  const size_t fixed = cs::smem_bytes_cs(threads, 0);
  const size_t budget = smem_per_block(kBlocks * (kThreads / threads));
  const int nwarp = threads / 32;
  long long cap = budget > fixed ? (long long)((budget - fixed) / (4 * (size_t)nwarp)) : 0;
  const long long most = (long long)n_steps * 64 * Granule<TIn>::kElems;
  if (cap > most) cap = most;
  if (cap < 32 * Granule<TIn>::kElems) return cudaErrorNotSupported;
  const size_t smem = cs::smem_bytes_cs(threads, (int)cap);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  k<<<(unsigned)p.T, threads, smem, s>>>(p, n_steps, (int)cap);
  return cudaGetLastError();
}

template <typename TIn, typename TGrad>
static cudaError_t launch_rows(const RowParams &p, uint32_t hint, cudaStream_t s) {
  constexpr int kElems = Granule<TIn>::kElems;
  int threads = hint & 0xffff, stage = (hint >> 16) & 0xff, cluster = (hint >> 24) & 0xff;
  const int stage_hint = stage;
  // stage byte 0x11: the kernel that keeps the row in shared memory; 0x1e: the same with
  // block 0's first copy withheld (self-test of the wait limit)
  if ((stage == 0x11 || stage == 0x1e) && !p.given_logp_mp_i) {
    const bool ok16 = aligned32(p.train, p.ld_train, sizeof(TIn)) &&
                      aligned32(p.infer, p.ld_infer, sizeof(TIn)) &&
                      aligned32(p.grad, p.ld_grad, sizeof(TGrad));
    const cudaError_t e =
        ok16 ? res::launch_resident<TIn, TGrad>(p, s, stage == 0x1e) : cudaErrorNotSupported;
    if (e != cudaErrorNotSupported) return e;
    cluster = 0;  // rows it cannot take: the streaming kernel below
  }
  // measured on B200: 4-byte logits run best with 2 x 512 threads per SM, 2-byte
  // logits (twice the exponentials per byte) with 4 x 256
  if (threads == 0) threads = sizeof(TIn) == 4 ? 512 : 256;
  stage = 2;  // two granules per thread and pipeline stage
  const bool vec_ok = aligned32(p.train, p.ld_train, sizeof(TIn)) &&
                      aligned32(p.infer, p.ld_infer, sizeof(TIn)) &&
                      aligned32(p.grad, p.ld_grad, sizeof(TGrad));
  const long long n_gran_row = (p.V + kElems - 1) / kElems;
  if (cluster == 0) cluster = 1;
  const bool weighted = p.weight_kind != DVP_WEIGHT_NONE;  // one block per row only
  if (weighted) cluster = 1;
  if (cluster > 1 && (n_gran_row < 4096 || p.T * cluster > 0x7fffffffLL)) cluster = 1;
  const long long n_gran = (n_gran_row + cluster - 1) / cluster;  // granules per block
  // shrink the block for short rows so that threads are not idle
  while (threads > 64 && (long long)threads * stage / 2 >= n_gran) threads /= 2;
  const long long per = (long long)stage * threads;
  const size_t smem = (size_t)smem_words_fixed(threads) * 4 +
                      (size_t)((n_gran + per - 1) / per) * per * sizeof(uint16_t);
  // 16-bit hot-list entries hold slot * 32 + lane: very long rows swept by few threads
  // would not fit them
  const bool hot_ok = ((n_gran + per - 1) / per) * stage * 32 <= 65536;
  if constexpr (sizeof(TIn) == 2) {
    // stage byte 3 or 4: the kernel that keeps the candidates of the safe set on chip, with
    // three or four resident blocks per SM (measured slower than the kernel below; kept for
    // comparison)
    if (vec_ok && cluster == 1 && (stage_hint == 3 || stage_hint == 4) && threads <= 256) {
      const int n_steps = (int)((n_gran + per - 1) / per);
      cudaError_t e;
      if (weighted)
        e = launch_rows_cs<TIn, TGrad, 256, 3, true>(p, threads, n_steps, s);
      else if (stage_hint == 3)
        e = launch_rows_cs<TIn, TGrad, 256, 3, false>(p, threads, n_steps, s);
      else
        e = launch_rows_cs<TIn, TGrad, 256, 4, false>(p, threads, n_steps, s);
      if (e != cudaErrorNotSupported) return e;
    }
  }
  if (vec_ok && hot_ok && smem <= 200 * 1024) {
    if (cluster == 4 && threads <= 256 && stage == 2)
      return launch_rows_vec<TIn, TGrad, 2, 256, 4, 4>(p, threads, smem, s);
    if (cluster == 2 && threads <= 256 && stage == 2)
      return launch_rows_vec<TIn, TGrad, 2, 256, 4, 2>(p, threads, smem, s);
    if (weighted) {
      if (threads > 256) return launch_rows_vec<TIn, TGrad, 2, 512, 2, 1, true>(p, threads, smem, s);
      return launch_rows_vec<TIn, TGrad, 2, 256, 4, 1, true>(p, threads, smem, s);
    }
    if (threads > 256) return launch_rows_vec<TIn, TGrad, 2, 512, 2, 1>(p, threads, smem, s);
    return launch_rows_vec<TIn, TGrad, 2, 256, 4, 1>(p, threads, smem, s);
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

template <typename TIn, typename TGrad>
static cudaError_t launch_bwd(const BackwardParams &p, uint32_t hint, cudaStream_t s) {
  int threads = hint & 0xffff;
  if (threads == 0) threads = 256;
  const bool vec_ok =
      aligned32(p.train, p.ld_train, sizeof(TIn)) && aligned32(p.grad, p.ld_grad, sizeof(TGrad));
  if (vec_ok)
    dvp_backward_kernel<TIn, TGrad, 2, true><<<(unsigned)p.T, threads, 0, s>>>(p);
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

}  // namespace dvp
