// Row kernel that keeps (most of) the row on chip (sm_100a).
//
// The threshold of Def. 5.1 needs the maximum of the whole row before any token
// can be masked, so a row has to be looked at twice (three times with the
// gradient of Prop. 5.4).  One block owns one row at a time and the second and
// third look are served from shared memory and L2 instead of HBM:
//
//   * the row is cut into slots of 30 KB (four 16-byte vectors per consumer thread).
//     The last R slots of a row stay in a "resident" ring of shared memory from the
//     first sweep to the last one that needs them; the first n - R slots pass
//     through a small "stream" ring, once for sweep 1 (from HBM) and once for
//     sweep 2 (from L2: a block re-reads what it read a few microseconds earlier).
//     Rows of up to 120 KB are resident as a whole.
//   * a producer warp issues every bulk copy, in the one order both sides know:
//     per matrix ("side") of a token the streamed slots, the resident slots, the
//     streamed slots again for sweep 2; then the next side.  Each copy completes
//     on its slot's "full" mbarrier and may be issued once the slot's "empty"
//     mbarrier says that every consumer warp is done with the previous content,
//     so the producer runs ahead of the consumers by whatever the rings have free,
//     across sweeps, sides and tokens.
//   * 15 consumer warps: sweep 1 (A1, A3) online log-sum-exp and maximum;
//     block reduction -> threshold (A2); sweep 2 (A4) masked sum and count, only
//     elements at or above the threshold cost more than a packed compare, and
//     each thread flags its vectors that hold a safe token; block reduction ->
//     per-token results (A5, A6); sweep 3 (A7) writes zeros for unflagged vectors
//     without reading anything and revisits the flagged ones (resident slot, or L2).
//
// HBM sees each logit once, whatever the density of the safe set.  Measured, it is
// slower than the streaming kernel (one row per SM runs its phases one after
// another); it is kept as an option behind the launch hint.  The kernel is
// persistent: block b takes tokens b, b + grid, ...
//
// Every mbarrier wait is bounded.  A wait that runs out sets an abort word in
// shared memory and a status word in global memory; from then on every wait
// of the block returns at once and stores are suppressed, the control flow stays
// the same and the kernel ends in bounded time.
#pragma once
#include <type_traits>

#include "dvp_common.cuh"

namespace dvp {
namespace res {

// 15 consumer warps and the producer warp: four warps per SM sub-partition, so
// that each thread may hold up to 128 registers
constexpr int kConsumerWarps = 15;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kThreads = kConsumers + 32;  // + the producer warp
constexpr int kMaxSlots = 64;
// Polls of one wait.  A poll may suspend the thread for up to kSuspendNs (the hint given
// to try_wait) and is followed by a 40 ns sleep: a wait gives up after about a second.
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr uint32_t kSuspendNs = 200;

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kSuspendNs)
      : "memory");
  return ok != 0;
}
// Global -> shared bulk copy of `bytes` (a multiple of 16, both addresses 16-byte
// aligned) that completes on an mbarrier of this block.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(addr));
  return v;
}

// Control words of one block, at the start of its dynamic shared memory.
struct Control {
  unsigned long long full[kMaxSlots];   // per slot: the bulk copy has landed
  unsigned long long empty[kMaxSlots];  // per slot: every consumer warp is done with it
  unsigned long long xbar[2];           // block reductions, alternating
  volatile int abort;                   // a wait of this block ran out
  int pad_[3];
  float xbuf[2][16][4];                 // reduction slots: [parity][warp]
};

enum { kWaitFull = 1, kWaitEmpty = 2, kWaitReduce = 4 };

struct Waiter {
  volatile int *abort;
  unsigned int *status;  // global status word
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, int code) {
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
      if (mbar_try_wait(bar, parity)) return true;
      if (*abort) return false;
      if (it > 64) __nanosleep(40);
    }
    *abort = 1;
    atomicOr(status, (unsigned int)code);
    return false;
  }
};

// ---- one 16-byte vector of a row ------------------------------------------------

template <typename TIn>
struct Vec {
  static constexpr int kElems = 16 / (int)sizeof(TIn);
  uint4 r;

  __device__ __forceinline__ void get(float *x) const { Storage<TIn>::unpack(r, x); }

  __device__ __forceinline__ float max() const {
    if constexpr (sizeof(TIn) == 4) {
      return fmaxf(fmaxf(__uint_as_float(r.x), __uint_as_float(r.y)),
                   fmaxf(__uint_as_float(r.z), __uint_as_float(r.w)));
    } else {
      using T2 = typename Pair<TIn>::type;
      const T2 a = __hmax2(*reinterpret_cast<const T2 *>(&r.x), *reinterpret_cast<const T2 *>(&r.y));
      const T2 b = __hmax2(*reinterpret_cast<const T2 *>(&r.z), *reinterpret_cast<const T2 *>(&r.w));
      const T2 c = __hmax2(a, b);
      return fmaxf(Storage<TIn>::widen(c.x), Storage<TIn>::widen(c.y));
    }
  }
};

// The threshold in a form that one packed compare per 32-bit word can test.
// Stored values are of type TIn, so "x >= tau" (tau a float) holds exactly when
// x >= tau rounded up to TIn: no value of the type lies between the two.
//
// hits() returns one bit per element at or above the threshold, at position
// code_of(j) for element j of the vector; element_of() inverts it.
template <typename TIn>
struct PackedTau {
  static constexpr int kElems = 16 / (int)sizeof(TIn);
  uint32_t w;
  __device__ __forceinline__ explicit PackedTau(float tau) {
    if constexpr (sizeof(TIn) == 4) {
      w = __float_as_uint(tau);
    } else if constexpr (std::is_same<TIn, __nv_bfloat16>::value) {
      const __nv_bfloat16 t = __float2bfloat16_ru(tau);
      const __nv_bfloat162 t2 = __halves2bfloat162(t, t);
      w = *reinterpret_cast<const uint32_t *>(&t2);
    } else {
      const __half t = __float2half_ru(tau);
      const __half2 t2 = __halves2half2(t, t);
      w = *reinterpret_cast<const uint32_t *>(&t2);
    }
  }
  __device__ __forceinline__ uint32_t hits(const uint4 &r) const {
    if constexpr (sizeof(TIn) == 4) {
      const float t = __uint_as_float(w);
      return (uint32_t)(__uint_as_float(r.x) >= t) | ((uint32_t)(__uint_as_float(r.y) >= t) << 1) |
             ((uint32_t)(__uint_as_float(r.z) >= t) << 2) | ((uint32_t)(__uint_as_float(r.w) >= t) << 3);
    } else {
      using T2 = typename Pair<TIn>::type;
      const T2 t2 = *reinterpret_cast<const T2 *>(&w);
      const uint32_t m0 = __hge2_mask(*reinterpret_cast<const T2 *>(&r.x), t2);
      const uint32_t m1 = __hge2_mask(*reinterpret_cast<const T2 *>(&r.y), t2);
      const uint32_t m2 = __hge2_mask(*reinterpret_cast<const T2 *>(&r.z), t2);
      const uint32_t m3 = __hge2_mask(*reinterpret_cast<const T2 *>(&r.w), t2);
      // bit i: low half of word i, bit 16 + i: high half of word i
      return (m0 & 0x00010001u) | (m1 & 0x00020002u) | (m2 & 0x00040004u) | (m3 & 0x00080008u);
    }
  }
  static __device__ __forceinline__ uint32_t code_of(int j) {
    if constexpr (sizeof(TIn) == 4) return 1u << j;
    else return 1u << ((j >> 1) + 16 * (j & 1));
  }
  static __device__ __forceinline__ int element_of(int bit) {
    if constexpr (sizeof(TIn) == 4) return bit;
    else return 2 * (bit & 15) + (bit >> 4);
  }
  static constexpr uint32_t kAll = sizeof(TIn) == 4 ? 0xfu : 0x000f000fu;
};

// Element j (a run-time index) of a vector held in registers.
template <typename TIn>
__device__ __forceinline__ float element(const uint4 &r, int j) {
  if constexpr (sizeof(TIn) == 4) {
    const uint32_t lo = (j & 1) ? r.y : r.x, hi = (j & 1) ? r.w : r.z;
    return __uint_as_float((j & 2) ? hi : lo);
  } else {
    const int wi = j >> 1;
    const uint32_t lo = (wi & 1) ? r.y : r.x, hi = (wi & 1) ? r.w : r.z;
    const uint32_t word = (wi & 2) ? hi : lo;
    const uint16_t bits = (uint16_t)((j & 1) ? (word >> 16) : (word & 0xffffu));
    if constexpr (std::is_same<TIn, __nv_bfloat16>::value) {
      return __uint_as_float((uint32_t)bits << 16);
    } else {
      return __half2float(__ushort_as_half(bits));
    }
  }
}

// ---- block-wide reductions over the consumer warps ---------------------------------
// Each warp reduces its lanes in a fixed order, lane 0 leaves the warp's partial
// in slot [warp] and arrives on the reduction barrier; every thread then reads the
// slots in index order.  Successive reductions alternate between two barriers and
// two sets of slots: a warp can be at most one reduction ahead of another.

struct Reducer {
  Control *ctl;
  Waiter w;
  uint32_t count;  // reductions done so far

  __device__ __forceinline__ void post(float a, float b, float c, float d) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t par = count & 1;
    if (lane == 0) {
      *reinterpret_cast<float4 *>(&ctl->xbuf[par][warp][0]) = make_float4(a, b, c, d);
      mbar_arrive(smem_u32(&ctl->xbar[par]));  // release: the store above is visible to waiters
    }
  }
  __device__ __forceinline__ float4 wait_and_read() {
    const uint32_t par = count & 1;
    w.wait(smem_u32(&ctl->xbar[par]), (count >> 1) & 1, kWaitReduce);
    const int lane = threadIdx.x & 31;
    const float4 e = *reinterpret_cast<const float4 *>(&ctl->xbuf[par][lane < kConsumerWarps ? lane : 0][0]);
    ++count;
    return e;
  }
};

__device__ __forceinline__ LogSum warp_reduce_logsum(LogSum v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    LogSum other;
    other.m = __shfl_xor_sync(0xffffffffu, v.m, o);
    other.c = __shfl_xor_sync(0xffffffffu, v.c, o);
    other.s = __shfl_xor_sync(0xffffffffu, v.s, o);
    v = (lane & o) ? combine(other, v) : combine(v, other);
  }
  return v;
}

__device__ __forceinline__ SumCount warp_reduce_sumcount(SumCount v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float os = __shfl_xor_sync(0xffffffffu, v.s, o);
    const int on = __shfl_xor_sync(0xffffffffu, v.n, o);
    v.s = (lane & o) ? os + v.s : v.s + os;
    v.n += on;
  }
  return v;
}

__device__ __forceinline__ LogSum block_logsum(Reducer &x, LogSum v) {
  v = warp_reduce_logsum(v);
  x.post(v.m, v.c, v.s, 0.f);
  const float4 e = x.wait_and_read();
  const bool mine = (threadIdx.x & 31) < kConsumerWarps;  // the other lanes repeat slot 0: left out
  LogSum r = {mine ? e.x : kNegInf, mine ? e.y : kNegInf, mine ? e.z : 0.f};
  return warp_reduce_logsum(r);
}

__device__ __forceinline__ SumCount block_sumcount(Reducer &x, SumCount v) {
  v = warp_reduce_sumcount(v);
  x.post(v.s, __int_as_float(v.n), 0.f, 0.f);
  const float4 e = x.wait_and_read();
  const bool mine = (threadIdx.x & 31) < kConsumerWarps;
  SumCount r = {mine ? e.x : 0.f, mine ? __float_as_int(e.y) : 0};
  return warp_reduce_sumcount(r);
}

// ---- how a row maps onto the two rings ---------------------------------------------

struct Geometry {
  int n_vec;     // 16-byte vectors in a row
  int n_chunks;  // slots a row takes
  int n_stream;  // leading slots that pass through the stream ring once per sweep
  int res_slots; // slots of the resident ring (slots 0 .. res_slots-1 of the block)
  int str_slots; // slots of the stream ring (the next str_slots slots)
};

struct Cursor {
  int slot;        // position within its ring
  uint32_t phase;  // parity of the slot's current use
  __device__ __forceinline__ void advance(int n_slots) {
    if (++slot == n_slots) {
      slot = 0;
      phase ^= 1;
    }
  }
};

struct ResidentParams {
  RowParams row;
  Geometry geo;
  unsigned int *status;  // global status word, OR-ed with kWait* codes
  int withhold_first;    // self-test: block 0 never issues its first copy, so its first wait runs out
};

// A slot holds kGroup 16-byte vectors per consumer thread (30 KB): one bulk copy, one
// wait and one hand-back per slot keep the cost of the barrier operations (a few
// hundred cycles each) small beside the work on a slot, and give every thread
// kGroup independent loads per step.  Thread `tid` owns vectors u * kConsumers + tid.
constexpr int kGroup = 4;
constexpr int kSlotVec = kGroup * kConsumers;
constexpr uint32_t kSlotBytes = (uint32_t)kSlotVec * 16u;
constexpr int kMaxChunks = 64 / kGroup;  // one flag bit per vector of a thread

// What the consumer warps of a block share while they walk the rings.
struct Walk {
  Control *ctl;
  uint32_t base;  // shared-memory address of slot 0
  Geometry geo;
  Cursor res, str;  // next use of the resident and of the stream ring
  Waiter w;

  __device__ __forceinline__ uint32_t slot_addr(int slot) const {
    if (!DVP_IN(slot, n_slot, DVP_OOB_SLOT)) slot = 0;  // bounds-checking build: reported, slot 0 read instead
    return base + (uint32_t)slot * kSlotBytes;
  }

  // Resident slot that holds chunk `ch` (>= n_stream) of the side whose resident part starts at `first`.
  __device__ __forceinline__ int resident_slot(const Cursor first, int ch) const {
    int s = first.slot + (ch - geo.n_stream);
    return s >= geo.res_slots ? s - geo.res_slots : s;
  }

  // One sweep over a row: the streamed slots as they land (each handed back at
  // once), then the resident slots starting at `first` (waited for in sweep 1,
  // handed back when `release_res`).  f(chunk, slot address).
  template <bool kWaitRes, class F>
  __device__ __forceinline__ void sweep(const Cursor first, bool release_res, F &&f) {
    const int lane = threadIdx.x & 31;
    Cursor r = first;
    for (int ch = 0; ch < geo.n_chunks; ++ch) {
      int slot, back = -1;  // back: the slot to hand back after this step
      if (ch < geo.n_stream) {
        slot = back = geo.res_slots + str.slot;
        w.wait(smem_u32(&ctl->full[slot]), str.phase, kWaitFull);
        str.advance(geo.str_slots);
      } else {
        slot = r.slot;
        if (kWaitRes) w.wait(smem_u32(&ctl->full[slot]), r.phase, kWaitFull);
        if (release_res) back = slot;
        r.advance(geo.res_slots);
      }
      f(ch, slot_addr(slot));
      if (back >= 0) {
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->empty[back]));
      }
    }
    if (kWaitRes) res = r;
  }
};

template <typename TIn>
__device__ __forceinline__ float lds_element(uint32_t addr) {
  if constexpr (sizeof(TIn) == 4) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
  } else {
    uint16_t b;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(b) : "r"(addr));
    if constexpr (std::is_same<TIn, __nv_bfloat16>::value) return __uint_as_float((uint32_t)b << 16);
    else return __half2float(__ushort_as_half(b));
  }
}

// Gradient entries of one vector (Prop. 5.4): coef * e^{x - m} at or above the
// threshold, 0 below, g_a at the sampled token (ja, or -1).
template <typename TIn, typename TGrad>
__device__ __forceinline__ void grad_vector(const uint4 &r, TGrad *dst, const PackedTau<TIn> &gtau, float m,
                                            float coef, int ja, float g_a) {
  constexpr int kElems = Vec<TIn>::kElems;
  using PT = PackedTau<TIn>;
  uint32_t code = gtau.hits(r);
  float out[kElems];
  if (code == PT::kAll) {
    float xs[kElems];
    Storage<TIn>::unpack(r, xs);
#pragma unroll
    for (int j = 0; j < kElems; ++j) out[j] = coef * ex2((xs[j] - m) * kLog2e);
  } else {
#pragma unroll
    for (int j = 0; j < kElems; ++j) out[j] = 0.f;
    while (code) {
      const int bit = __ffs(code) - 1;
      code &= code - 1;
      const int j = PT::element_of(bit);
      const float val = coef * ex2((element<TIn>(r, j) - m) * kLog2e);
#pragma unroll
      for (int jj = 0; jj < kElems; ++jj)
        if (jj == j) out[jj] = val;
    }
  }
#pragma unroll
  for (int jj = 0; jj < kElems; ++jj)
    if (jj == ja) out[jj] = g_a;
  store_grads<TGrad, kElems>(dst, out);
}

// Consumer side of one matrix ("side") of one token: sweeps 1 and 2, and sweep 3
// when a gradient row is asked for.  Returns the statistics of the row.
template <typename TIn, typename TGrad>
__device__ __forceinline__ SideStats consume_side(const TIn *row, TGrad *grow, float g, int V, int a,
                                                  const RowParams &p, Walk &wk, Reducer &red,
                                                  uint32_t *mask_row, const SideStats *other = nullptr,
                                                  float *weight = nullptr) {
  constexpr int kElems = Vec<TIn>::kElems;
  using PT = PackedTau<TIn>;
  const int tid = threadIdx.x, lane = tid & 31;
  const int n_vec = wk.geo.n_vec;
  const uint32_t my = (uint32_t)tid * 16u;  // this thread's vector within every slot
  volatile int *abort = wk.w.abort;

  const bool has_a = a >= 0 && a < V;
  // the sampled token's logit: one element, fetched while the row streams in
  const float z_a = has_a ? Storage<TIn>::widen(row[a]) : 0.f;
  const Cursor first = wk.res;

  // ---- sweep 1: maximum and log-sum-exp, as the row lands
  LogSum acc = {kNegInf, kNegInf, 0.f};
  wk.template sweep<true>(first, false, [&](int ch, uint32_t slot) {
    Vec<TIn> v[kGroup];
    bool valid[kGroup];
    float cm = kNegInf;
#pragma unroll
    for (int u = 0; u < kGroup; ++u) {
      valid[u] = ch * kSlotVec + u * kConsumers + tid < n_vec;
      if (valid[u]) v[u].r = lds128(slot + my + (uint32_t)u * kConsumers * 16u);
    }
#pragma unroll
    for (int u = 0; u < kGroup; ++u)
      if (valid[u]) cm = fmaxf(cm, v[u].max());
    if (cm > kNegInf) {
      if (cm > acc.m) {
        const float cn = cm * kLog2e;
        acc.s *= ex2(acc.c - cn);  // acc.c = -inf at the start: the factor is 0
        acc.m = cm;
        acc.c = cn;
      }
      const float neg_c = -acc.c;
      float part[kGroup];
#pragma unroll
      for (int u = 0; u < kGroup; ++u) {
        part[u] = 0.f;
        if (valid[u]) {
          float xs[kElems];
          v[u].get(xs);
#pragma unroll
          for (int j = 0; j < kElems; ++j) part[u] += ex2(fmaf(xs[j], kLog2e, neg_c));
        }
      }
      acc.s += (part[0] + part[1]) + (part[2] + part[3]);
    }
  });
  const LogSum all = block_logsum(red, acc);

  SideStats st;
  st.m = all.m;
  st.lse = lse_from_logsum(all);
  st.sum_c = (double)all.c;
  st.sum_s = all.s;
  st.tau = threshold_of<TIn>(all.m, p.log_rho, p.mode);
  st.z_a = z_a;
  st.member = has_a && z_a >= st.tau;
  st.e_a = st.member ? ex2((z_a - st.m) * kLog2e) : 0.f;

  // ---- sweep 2: masked sum without the sampled token, count, flags of the vectors
  // that hold a safe token (and the packed mask).  Elements below the threshold
  // cost a packed compare; the others are visited one by one, over the whole group.
  const bool has_grad = grow != nullptr;
  const PT ptau(st.tau);
  const int a_vec = has_a ? a / kElems : -1;  // vector of the row that holds a
  const uint32_t a_code = has_a ? PT::code_of(a % kElems) : 0u;
  const float m = st.m;  // e^{x - m} from the exact difference, as in the per-token results
  SumCount sc = {0.f, 0};
  unsigned long long flagged = 0;  // bit ch: this thread's vector of slot ch holds a safe token
  wk.template sweep<false>(first, !has_grad, [&](int ch, uint32_t slot) {
    uint4 r[kGroup];
    uint32_t code[kGroup];
    uint32_t merged = 0;
    bool dense = true;
#pragma unroll
    for (int u = 0; u < kGroup; ++u) {
      const int vi = ch * kSlotVec + u * kConsumers + tid;
      const bool valid = vi < n_vec;
      code[u] = 0;
      if (valid) {
        r[u] = lds128(slot + my + (uint32_t)u * kConsumers * 16u);
        code[u] = ptau.hits(r[u]);
      }
      sc.n += __popc(code[u]);
      if (code[u]) flagged |= 1ull << (ch * kGroup + u);
      const uint32_t rest = vi == a_vec ? code[u] & ~a_code : code[u];  // a is counted, not summed
      dense = dense && rest == PT::kAll;
      merged |= rest << (4 * u);
    }
    if (dense) {  // a dense safe set: no per-hit bookkeeping
#pragma unroll
      for (int u = 0; u < kGroup; ++u) {
        float xs[kElems];
        Storage<TIn>::unpack(r[u], xs);
#pragma unroll
        for (int j = 0; j < kElems; ++j) sc.s += ex2((xs[j] - m) * kLog2e);
      }
    } else {
      while (merged) {
        const int bit = __ffs(merged) - 1;
        merged &= merged - 1;
        int u, j;
        if constexpr (sizeof(TIn) == 4) {
          u = bit >> 2;
          j = bit & 3;
        } else {
          u = (bit & 15) >> 2;
          j = 2 * (bit & 3) + (bit >> 4);
        }
        const uint32_t ea = slot + my + (uint32_t)u * kConsumers * 16u + (uint32_t)j * (uint32_t)sizeof(TIn);
        sc.s += ex2((lds_element<TIn>(ea) - m) * kLog2e);
      }
    }
    if (mask_row) {  // uniform over the block: the lanes of one word meet by shuffles
      constexpr int kLanesPerWord = 32 / kElems;
#pragma unroll
      for (int u = 0; u < kGroup; ++u) {
        const int vi = ch * kSlotVec + u * kConsumers + tid;
        uint32_t bits = 0;
#pragma unroll
        for (int j = 0; j < kElems; ++j) bits |= (code[u] & PT::code_of(j)) ? 1u << j : 0u;
        uint32_t word = bits << (kElems * (lane % kLanesPerWord));
#pragma unroll
        for (int o = 1; o < kLanesPerWord; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
        if (vi < n_vec && lane % kLanesPerWord == 0 && !*abort)
          mask_row[vi / kLanesPerWord] = word;
      }
    }
  });
  const SumCount tot = block_sumcount(red, sc);
  st.s_x = tot.s;
  st.n = tot.n;
  set_mask_mass(st, V, p.mode, Storage<TIn>::widen(Storage<TIn>::narrow(p.mask_value)), has_a);

  // ---- sweep 3: the gradient row (Prop. 5.4, set fixed), to HBM.  Vectors without
  // a safe token are zeros and need no read; the flagged ones are read again from
  // their resident slot, or from global memory (L2) when they were streamed.
  const int n_res = wk.geo.n_chunks - wk.geo.n_stream;
  if (other) {  // the importance weight of this token, from both sides' statistics
    const float wt = row_weight(p, st, *other, has_a);
    *weight = wt;
    if (wt == wt) g *= wt;
  }
  if (has_grad) {
    const float s_tot = st.s_x + st.e_a + st.s_mask;
    const bool live = st.live;
    const float coef = live ? -g / s_tot : 0.f;
    const float g_a = st.member ? g * ((st.s_x + st.s_mask) / s_tot) : 0.f;
    const int av = (live && st.member) ? a_vec : -1;
    // a row without a gradient (sampled token missing or pruned) is all zeros
    if (!live) flagged = 0;
    const bool ok = !*abort;
    if (ok) {
      for (int ch = 0; ch < wk.geo.n_chunks; ++ch) {
#pragma unroll
        for (int u = 0; u < kGroup; ++u) {
          const int vi = ch * kSlotVec + u * kConsumers + tid;
          if (vi < n_vec && !((flagged >> (ch * kGroup + u)) & 1ull))
            store_zeros<TGrad, kElems>(grow + (size_t)vi * kElems);
        }
      }
      while (flagged) {
        const int bit = __ffsll((long long)flagged) - 1;
        flagged &= flagged - 1;
        const int ch = bit / kGroup, u = bit % kGroup;
        const int vi = ch * kSlotVec + u * kConsumers + tid;
        uint4 r;
        if (ch >= wk.geo.n_stream)
          r = lds128(wk.slot_addr(wk.resident_slot(first, ch)) + my + (uint32_t)u * kConsumers * 16u);
        else r = ld_stream16(reinterpret_cast<const char *>(row) + (size_t)vi * 16);
        grad_vector<TIn, TGrad>(r, grow + (size_t)vi * kElems, ptau, m, coef, vi == av ? a % kElems : -1, g_a);
      }
    }
    // the resident slots go back to the producer
    __syncwarp();
    if (lane == 0) {
      Cursor r = first;
      for (int i = 0; i < n_res; ++i) {
        mbar_arrive(smem_u32(&wk.ctl->empty[r.slot]));
        r.advance(wk.geo.res_slots);
      }
    }
  }
  return st;
}

// Shared memory of one block: the control words, then the slots (128-byte aligned).
__host__ __device__ constexpr size_t control_bytes() { return (sizeof(Control) + 127) & ~(size_t)127; }

template <typename TIn, typename TGrad>
__global__ void __launch_bounds__(kThreads, 1) dvp_row_kernel_resident(const ResidentParams rp) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Control *ctl = reinterpret_cast<Control *>(smem_raw);
  const uint32_t base = smem_u32(smem_raw + control_bytes());

  const RowParams &p = rp.row;
  const Geometry geo = rp.geo;
  const int V = (int)p.V;
  const bool two_sides = p.infer != nullptr;
  // with an importance weight the gradient needs the inference side's result first
  const bool infer_first = two_sides && p.weight_kind != DVP_WEIGHT_NONE;
  const int n_slots = geo.res_slots + geo.str_slots;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_slots; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), kConsumerWarps);
    }
    mbar_init(smem_u32(&ctl->xbar[0]), kConsumerWarps);
    mbar_init(smem_u32(&ctl->xbar[1]), kConsumerWarps);
    ctl->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  DVP_BOUNDS_BEGIN(p.bounds_status);
  DVP_BOUNDS_SET(n_slot, n_slots);
  DVP_BOUNDS_SET(V, geo.n_vec);  // this kernel counts a row in 16-byte vectors
  DVP_BOUNDS_SYNC();

  Waiter w = {&ctl->abort, rp.status};

  if (threadIdx.x >= kConsumers) {
    // ---- producer: one lane issues every copy, in the order the consumers expect
    if (threadIdx.x == kConsumers) {
      Cursor res = {0, 0}, str = {0, 0};
      bool ok = true;
      // Copies slot `ch` of a row into the next slot of a ring; false once a wait ran out.
      bool withhold = rp.withhold_first != 0 && blockIdx.x == 0;
      auto issue = [&](const char *row_bytes, int ch, Cursor &cur, int ring_first, int ring_slots) {
        const int slot = ring_first + cur.slot;
        if (withhold) {  // the slot is taken but nothing will ever land in it
          withhold = false;
          cur.advance(ring_slots);
          return true;
        }
        // the slot's previous use is over (a fresh barrier passes the first time round)
        if (!w.wait(smem_u32(&ctl->empty[slot]), cur.phase ^ 1, kWaitEmpty)) return false;
        if (*w.abort) return false;  // consumers no longer wait for what is issued
        const int left = geo.n_vec - ch * kSlotVec;
        const uint32_t bytes = (uint32_t)(left < kSlotVec ? left : kSlotVec) * 16u;
        const uint32_t bar = smem_u32(&ctl->full[slot]);
        // bounds-checking build: a copy outside the slots or past the row is reported and not issued
        // (the wait for it then runs out and ends the launch, which is reported as well)
        if (!DVP_IN(slot, n_slot, DVP_OOB_SLOT) ||
            !DVP_IN((long long)ch * kSlotVec + (long long)bytes / 16 - 1, V, DVP_OOB_GLOBAL)) {
          cur.advance(ring_slots);
          return true;
        }
        mbar_expect_tx(bar, bytes);
        bulk_load(base + (uint32_t)slot * kSlotBytes, row_bytes + (size_t)ch * kSlotBytes, bytes, bar);
        cur.advance(ring_slots);
        return true;
      };
      for (long long t = blockIdx.x; t < p.T && ok; t += gridDim.x) {
        for (int side = 0; side < (two_sides ? 2 : 1) && ok; ++side) {
          const bool train_side = (side == 0) != infer_first;
          const TIn *row = train_side ? reinterpret_cast<const TIn *>(p.train) + t * p.ld_train
                                      : reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer;
          const char *src = reinterpret_cast<const char *>(row);
          for (int ch = 0; ch < geo.n_stream && ok; ++ch)  // sweep 1, streamed part
            ok = issue(src, ch, str, geo.res_slots, geo.str_slots);
          for (int ch = geo.n_stream; ch < geo.n_chunks && ok; ++ch)  // resident part
            ok = issue(src, ch, res, 0, geo.res_slots);
          for (int ch = 0; ch < geo.n_stream && ok; ++ch)  // sweep 2, streamed part again
            ok = issue(src, ch, str, geo.res_slots, geo.str_slots);
        }
      }
      if (!ok) {
        // let the copies still in flight land before this block's memory goes away
        for (uint32_t it = 0; it < 2000; ++it) __nanosleep(500);
      }
    }
    __syncwarp();
  } else {
    // ---- consumers
    Reducer red = {ctl, w, 0u};
    Walk wk = {ctl, base, geo, {0, 0}, {0, 0}, w};
    const size_t mask_words = (size_t)((p.V + 31) / 32);
    for (long long t = blockIdx.x; t < p.T; t += gridDim.x) {
      const long long id = p.ids ? load_id(p.ids, p.id_is_i32, t) : -1;
      const bool has_id = id >= 0, bad_id = id >= p.V;
      const int a = (has_id && !bad_id) ? (int)id : -1;

      const TIn *trow = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
      const TIn *irow = two_sides ? reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer : nullptr;
      TGrad *grow = p.grad ? reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad : nullptr;
      const float g = p.grad ? p.upstream[t] : 0.f;
      uint32_t *mask_t = p.out_t.mask ? p.out_t.mask + t * mask_words : nullptr;
      uint32_t *mask_i = p.out_i.mask ? p.out_i.mask + t * mask_words : nullptr;
      SideStats st, si;
      float wgt = 1.f;
      // one call site for both matrices: the second copy of the sweeps would cost registers
      for (int k = 0; k < (two_sides ? 2 : 1); ++k) {
        const bool train_side = (k == 0) != infer_first;
        // sweep 3 needs the weight between sweeps 2 and 3 of the training side: the callee
        // forms it from both sides' statistics
        const SideStats r = consume_side<TIn, TGrad>(
            train_side ? trow : irow, train_side ? grow : (TGrad *)nullptr, train_side ? g : 0.f, V, a, p, wk,
            red, train_side ? mask_t : mask_i, (train_side && infer_first) ? &si : nullptr, &wgt);
        if (train_side) st = r;
        else si = r;
      }
      if (p.weight_out && threadIdx.x == 0 && !ctl->abort) p.weight_out[t] = wgt;
      if (threadIdx.x == 0 && !ctl->abort) {
        const float lt = finish_side(p.out_t, t, st, has_id, bad_id);
        uint8_t flags = (uint8_t)((st.member ? DVP_FLAG_IN_TRAIN : 0) | (has_id ? 0 : DVP_FLAG_NO_ID) |
                                  (bad_id ? DVP_FLAG_BAD_ID : 0));
        if (two_sides) {
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
  }
}

// ---- host side ---------------------------------------------------------------------

// Device address of the library's status word for the current device (dvp_rows.cu).
unsigned int *row_status_word();

constexpr size_t kMaxDynamicSmem = 227 * 1024;
constexpr int kStreamSlots = 3;  // slots of the stream ring when a row is not resident as a whole

// Geometry for rows of `row_bytes` bytes; n_chunks = 0 when the kernel cannot take them.
static inline Geometry geometry_of(long long row_bytes) {
  Geometry g = {};
  size_t total = (kMaxDynamicSmem - control_bytes()) / kSlotBytes;
  if (total > (size_t)kMaxSlots) total = kMaxSlots;
  if (row_bytes <= 0 || row_bytes % 16 != 0) return g;
  const long long n = (row_bytes / 16 + kSlotVec - 1) / kSlotVec;
  if (n > kMaxChunks) return g;
  g.n_vec = (int)(row_bytes / 16);
  if (n + kStreamSlots <= (long long)total) {  // the whole row resident, the other slots run ahead
    g.res_slots = (int)total;
    g.str_slots = 0;
    g.n_stream = 0;
  } else {
    g.str_slots = kStreamSlots;
    g.res_slots = (int)total - kStreamSlots;
    g.n_stream = (int)n - g.res_slots;
  }
  g.n_chunks = (int)n;
  return g;
}

template <typename TIn, typename TGrad>
static cudaError_t launch_resident(const RowParams &p, cudaStream_t s, bool withhold_first = false) {
  const Geometry geo = geometry_of(p.V * (long long)sizeof(TIn));
  if (geo.n_chunks == 0) return cudaErrorNotSupported;
  auto k = dvp_row_kernel_resident<TIn, TGrad>;
  const size_t smem = control_bytes() + (size_t)(geo.res_slots + geo.str_slots) * kSlotBytes;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  unsigned int *status = row_status_word();
  if (!status) return cudaErrorUnknown;
  int dev = 0, sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  ResidentParams rp;
  rp.row = p;
  rp.geo = geo;
  rp.status = status;
  rp.withhold_first = withhold_first ? 1 : 0;
  const unsigned grid = (unsigned)(p.T < (long long)sms ? p.T : (long long)sms);  // one block per SM
  k<<<grid, kThreads, smem, s>>>(rp);
  return cudaGetLastError();
}

}  // namespace res
}  // namespace dvp
