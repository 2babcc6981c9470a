// Row kernel for 2-byte logits that keeps the candidates of the safe set on chip.
//
// The threshold of Def. 5.1 needs the row maximum, which is known only when the
// whole row has been seen.  But the maximum seen so far can only grow, so
// "maximum so far + ln rho" never exceeds the final threshold: a logit below it
// can be dropped for good while the row still streams.  The running bound is one
// shared word that starts at the sampled token's logit (the row maximum or close
// to it in most rows) and that a thread raises with an atomic maximum when a
// granule of its own lifts it.
//
// During the one sweep over the row a lane whose 32-byte granule reaches the
// bound only copies the granule, as loaded, and its ordinal into a small ring of
// its warp (one ballot, three stores: lanes with such a granule are few, so
// anything longer would run with most of the warp idle).  When 32 granules have
// gathered, the warp takes one each and appends every element that reaches the
// bound, value and position in 4 bytes, to the warp's list in shared memory.
// Once the row maximum is known, the masked sum and the count of Def. 5.2 walk the
// list against the exact threshold, and the gradient of Prop. 5.4 is a row of
// zeros into which the safe entries of the list are scattered.  Nothing is read
// from global memory a second time.
//
// A warp whose list is full first drops the entries that the bound has overtaken;
// if that frees nothing it gives the list up and sweeps its share of the row a
// second and third time in global memory (dense safe sets end here).  Which warps
// do so depends on timing; the results do not: the masked sum is accumulated in
// fixed point, where addition is exact, so it does not depend on the order or on
// the path that supplied the terms.
#pragma once

namespace dvp {
namespace cs {

// Key of a float whose unsigned order is the float order.
__device__ __forceinline__ uint32_t float_key(float v) {
  const uint32_t b = __float_as_uint(v);
  return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  return __uint_as_float(k ^ ((k >> 31) ? 0x80000000u : 0xffffffffu));
}
__device__ __forceinline__ unsigned long long run_word(float v, uint32_t granule) {
  return ((unsigned long long)float_key(v) << 32) | granule;
}

// Largest value of the logits' type that is <= v.
template <typename TIn>
struct Below;
template <>
struct Below<__nv_bfloat16> {
  static __device__ __forceinline__ __nv_bfloat16 of(float v) {
    return __float2bfloat16_rz(bf16_round_down(v));  // exact: already a bfloat16 value
  }
};
template <>
struct Below<__half> {
  static __device__ __forceinline__ __half of(float v) { return __float2half_rd(v); }
};

__device__ __forceinline__ uint32_t ge2_mask(uint32_t w, __nv_bfloat162 t) {
  return __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&w), t);
}
__device__ __forceinline__ uint32_t ge2_mask(uint32_t w, __half2 t) {
  return __hge2_mask(*reinterpret_cast<const __half2 *>(&w), t);
}
__device__ __forceinline__ __nv_bfloat162 pair_of(__nv_bfloat16 v) { return __halves2bfloat162(v, v); }
__device__ __forceinline__ __half2 pair_of(__half v) { return __halves2half2(v, v); }

template <typename TIn>
__device__ __forceinline__ float widen_bits(uint16_t b) {
  return Storage<TIn>::widen(*reinterpret_cast<const TIn *>(&b));
}

constexpr int kRing = 96;  // staged granules per warp: up to 31 left over plus two appends of 32
constexpr int kRingBytes = kRing * 34;  // per warp

// ---- exact accumulation of e^{z - m} over the safe set --------------------------
// Terms lie in (0, 1].  Terms of 2^-22 and above are added as integers in units of
// 2^-kFixHi, smaller ones in units of 2^-(kFixHi + 23); a term is truncated to its unit,
// which loses nothing for terms above 2^(23 - kFixHi - 23) and at most one unit below.
// Integer addition is associative: the sums do not depend on the order of the terms.
constexpr int kFixHi = 40;  // up to 2^23 terms of at most 1.0 fit 64 bits
struct FixSum {
  unsigned long long hi, lo;
  int n;
};
__device__ __forceinline__ void fix_add(FixSum &f, float e) {
  if (e >= 0x1p-22f)
    f.hi += __float2ull_rz(e * 0x1p40f);
  else
    f.lo += __float2ull_rz(e * 0x1p63f);
}
__device__ __forceinline__ float fix_value(const FixSum &f) {
  return (float)((double)f.hi * 0x1p-40 + (double)f.lo * 0x1p-63);
}

// scratch: 160 words of shared memory.  Result valid in every thread.
__device__ __forceinline__ FixSum block_reduce_fix(FixSum v, float *scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    v.hi += __shfl_xor_sync(0xffffffffu, v.hi, o);
    v.lo += __shfl_xor_sync(0xffffffffu, v.lo, o);
    v.n += __shfl_xor_sync(0xffffffffu, v.n, o);
  }
  unsigned long long *s64 = reinterpret_cast<unsigned long long *>(scratch);
  int *s32 = reinterpret_cast<int *>(scratch) + 128;
  __syncthreads();  // scratch may still be read from an earlier reduction
  if (lane == 0) {
    s64[warp] = v.hi;
    s64[32 + warp] = v.lo;
    s32[warp] = v.n;
  }
  __syncthreads();
  FixSum r;
  r.hi = lane < nwarp ? s64[lane] : 0ull;
  r.lo = lane < nwarp ? s64[32 + lane] : 0ull;
  r.n = lane < nwarp ? s32[lane] : 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    r.hi += __shfl_xor_sync(0xffffffffu, r.hi, o);
    r.lo += __shfl_xor_sync(0xffffffffu, r.lo, o);
    r.n += __shfl_xor_sync(0xffffffffu, r.n, o);
  }
  return r;
}

// ---- the candidates of one warp ---------------------------------------------------
// A granule of the warp has the ordinal slot * 32 + lane (slot: which of its lane's
// granules); an element of it the position ordinal * 16 + element.  A list entry holds the
// element's 16 stored bits in its upper half and the position in its lower half.
struct WarpCand {
  uint32_t *list;  // this warp's list
  uint4 *ring;     // this warp's staged granules: kRing slots of 32 bytes, then kRing 16-bit ordinals
  int cap;         // entries the list holds
  int cnt;         // entries in use; negative: the list was given up
  int staged;      // ordinals in the ring
  float tb_tried;  // bound at the last attempt to make room
};

// Drops the list entries below `tb`, keeping the order of the others.
template <typename TIn>
__device__ __forceinline__ void drop_below(WarpCand &wc, float tb) {
  const int lane = threadIdx.x & 31;
  int kept = 0;
  for (int base = 0; base < wc.cnt; base += 32) {
    const bool valid = base + lane < wc.cnt;
    const uint32_t e = valid ? wc.list[base + lane] : 0u;
    const bool stay = valid && widen_bits<TIn>((uint16_t)(e >> 16)) >= tb;
    const uint32_t bal = __ballot_sync(0xffffffffu, stay);
    __syncwarp();  // every lane has read its entry before any lane overwrites one
    if (stay && DVP_IN(kept + __popc(bal & ((1u << lane) - 1u)), n_list, DVP_OOB_LIST))
      wc.list[kept + __popc(bal & ((1u << lane) - 1u))] = e;
    kept += __popc(bal);
  }
  __syncwarp();
  wc.cnt = kept;
}

__device__ __forceinline__ uint16_t *ring_ordinals(uint4 *ring) {
  return reinterpret_cast<uint16_t *>(ring + 2 * kRing);
}

// The warp takes the last `n` (<= 32) staged granules, one per lane, and appends their elements
// at or above `tb` to the list.
template <typename TIn>
__device__ __forceinline__ void drain(float tb, int n, WarpCand &wc) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int lane = threadIdx.x & 31;
  __syncwarp();  // what other lanes staged is visible
  wc.staged -= n;
  const int slot = wc.staged + lane;
  const bool valid = lane < n && DVP_IN(slot, n_ring, DVP_OOB_RING);
  const uint16_t *vals = reinterpret_cast<const uint16_t *>(wc.ring + 2 * slot);
  uint32_t ord = 0, k = 0;
  if (valid) {
    ord = ring_ordinals(wc.ring)[slot];
    const uint4 lo = wc.ring[2 * slot], hi = wc.ring[2 * slot + 1];
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    const auto t2 = pair_of(Below<TIn>::of(tb));
#pragma unroll
    for (int i = 0; i < 8; ++i) k |= ge2_mask(w[i], t2) & (0x00010001u << i);
    k = (k & 0xffu) | ((k >> 8) & 0xff00u);  // bit b: element 2 (b & 7) + (b >> 3)
  }
  const int nl = __popc(k);
  int incl = nl;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  const int total = __shfl_sync(0xffffffffu, incl, 31);
  if (wc.cnt + total > wc.cap) {
    // entries kept under an older, lower bound may have been overtaken
    if (tb > wc.tb_tried) {
      drop_below<TIn>(wc, tb);
      wc.tb_tried = tb;
    }
    if (wc.cnt + total > wc.cap) wc.cnt = -1;
  }
  if (wc.cnt >= 0) {
    uint32_t *dst = wc.list + wc.cnt + incl - nl;
    wc.cnt += total;
    while (k) {
      const int b = __ffs(k) - 1;
      k &= k - 1;
      const int j = 2 * (b & 7) + (b >> 3);
      if (DVP_IN(dst - wc.list, n_list, DVP_OOB_LIST)) *dst = ((uint32_t)vals[j] << 16) | (ord * kElems + (uint32_t)j);
      ++dst;
    }
  }
  __syncwarp();  // the slots are free again
}

// One pipeline stage of the sweep: log-sum-exp state as in absorb_stage; granules that reach
// the running bound are staged for the warp.
template <typename TIn>
__device__ __forceinline__ void absorb_stage_cs(const TIn *row, int V, const Stage<TIn, 2> &st, int step,
                                                LogSum &acc, WarpCand &wc, unsigned long long *run,
                                                float log_rho_dn) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int lane = threadIdx.x & 31;
  const float g0 = st.g[0].max(), g1 = st.g[1].max();
  const float cm = fmaxf(g0, g1);
  // the shared word holds the bound itself (as a key), not the maximum: readers need no arithmetic
  float tb = key_float(reinterpret_cast<volatile uint32_t *>(run)[1]);
  if (__fadd_rd(cm, log_rho_dn) > tb) {
    // never above the final threshold: the maximum only grows, both roundings go down
    const float mine = Storage<TIn>::widen(Below<TIn>::of(__fadd_rd(cm, log_rho_dn)));
    if (mine > tb) {
      const uint32_t gi = (uint32_t)((step * 2 + (g1 > g0 ? 1 : 0)) * (int)blockDim.x + (int)threadIdx.x);
      atomicMax(run, ((unsigned long long)float_key(mine) << 32) | gi);
      tb = mine;
    }
  }
  if (wc.cnt >= 0) {
    const bool hot0 = g0 >= tb, hot1 = g1 >= tb;
    const uint32_t bal0 = __ballot_sync(0xffffffffu, hot0), bal1 = __ballot_sync(0xffffffffu, hot1);
    if (bal0 | bal1) {
      const uint32_t below = (1u << lane) - 1u;
      if (hot0 && DVP_IN(wc.staged + __popc(bal0 & below), n_ring, DVP_OOB_RING)) {
        const int slot = wc.staged + __popc(bal0 & below);
        wc.ring[2 * slot] = make_uint4(st.g[0].w[0], st.g[0].w[1], st.g[0].w[2], st.g[0].w[3]);
        wc.ring[2 * slot + 1] = make_uint4(st.g[0].w[4], st.g[0].w[5], st.g[0].w[6], st.g[0].w[7]);
        ring_ordinals(wc.ring)[slot] = (uint16_t)(step * 64 + lane);
      }
      wc.staged += __popc(bal0);
      if (hot1 && DVP_IN(wc.staged + __popc(bal1 & below), n_ring, DVP_OOB_RING)) {
        const int slot = wc.staged + __popc(bal1 & below);
        wc.ring[2 * slot] = make_uint4(st.g[1].w[0], st.g[1].w[1], st.g[1].w[2], st.g[1].w[3]);
        wc.ring[2 * slot + 1] = make_uint4(st.g[1].w[4], st.g[1].w[5], st.g[1].w[6], st.g[1].w[7]);
        ring_ordinals(wc.ring)[slot] = (uint16_t)(step * 64 + 32 + lane);
      }
      wc.staged += __popc(bal1);
    }
  }

  if (cm > kNegInf) {
    if (cm > acc.m) {
      const float cn = cm * kLog2e;
      acc.s *= ex2(acc.c - cn);
      acc.m = cm;
      acc.c = cn;
    }
    const float neg_c = -acc.c;
    float part[4] = {0.f, 0.f, 0.f, 0.f};  // four chains: the additions do not wait on one another
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      float x[kElems];
      st.g[u].get(x);
#pragma unroll
      for (int j = 0; j < kElems; ++j) part[j & 3] += ex2(fmaf(x[j], kLog2e, neg_c));
    }
    acc.s += (part[0] + part[1]) + (part[2] + part[3]);
  }
}

// Takes batches of 32 staged ordinals while there are that many.
template <typename TIn>
__device__ __forceinline__ void drain_full(const TIn *row, int V, unsigned long long *run, WarpCand &wc) {
  if (wc.cnt < 0 || wc.staged < 32) return;
  const float tb = key_float(reinterpret_cast<volatile uint32_t *>(run)[1]);
#pragma unroll 1
  while (wc.staged >= 32) drain<TIn>(tb, 32, wc);
}

// The sweep over the row: one stage in flight while the previous one is absorbed.
template <typename TIn>
__device__ __forceinline__ LogSum sweep1_cs(const TIn *row, int V, int n_steps, WarpCand &wc,
                                            unsigned long long *run, float log_rho_dn, float *scratch) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int n_full = V / kElems;
  LogSum acc = {kNegInf, kNegInf, 0.f};
  if (n_steps > 0) {
    Stage<TIn, 2> s0, s1;
    s0.load(row, V, n_full, 0);
    int step = 0;
#pragma unroll 1
    for (; step + 1 < n_steps; step += 2) {
      s1.load(row, V, n_full, step + 1);
      absorb_stage_cs<TIn>(row, V, s0, step, acc, wc, run, log_rho_dn);
      // drained here, where only one stage's registers are live
      drain_full<TIn>(row, V, run, wc);
      if (step + 2 < n_steps) s0.load(row, V, n_full, step + 2);
      absorb_stage_cs<TIn>(row, V, s1, step + 1, acc, wc, run, log_rho_dn);
      drain_full<TIn>(row, V, run, wc);
    }
    if (step < n_steps) absorb_stage_cs<TIn>(row, V, s0, step, acc, wc, run, log_rho_dn);
  }
  drain_full<TIn>(row, V, run, wc);
  if (wc.cnt >= 0 && wc.staged > 0) {
    const float tb = key_float(reinterpret_cast<volatile uint32_t *>(run)[1]);
    drain<TIn>(tb, wc.staged, wc);
  }
  return block_reduce_logsum(acc, scratch);
}

// Position (in the numbering of WarpCand) of element `a` of the row if this warp owns it, else -1.
__device__ __forceinline__ int position_in_warp(int a, int kElems) {
  if (a < 0) return -1;
  const int nt = blockDim.x, g = a / kElems;
  const int owner = g % nt, slot = g / nt;
  if ((owner >> 5) != ((int)threadIdx.x >> 5)) return -1;
  return (slot * 32 + (owner & 31)) * kElems + a % kElems;
}

// Masked sum without the sampled token and count (Def. 5.2) of this warp's share of the row:
// from the list, or from global memory for a warp that gave its list up.
template <typename TIn>
__device__ __forceinline__ FixSum walk_sum(const TIn *row, int V, int n_steps, int a, float tau, float m,
                                           const WarpCand &wc) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int nt = blockDim.x, tid = threadIdx.x, lane = tid & 31;
  FixSum f = {0ull, 0ull, 0};
  if (wc.cnt >= 0) {
    const uint32_t pos_a = (uint32_t)position_in_warp(a, kElems);
    for (int i = lane; i < wc.cnt; i += 32) {
      if (!DVP_IN(i, n_list, DVP_OOB_LIST)) break;
      const uint32_t e = wc.list[i];
      const float x = widen_bits<TIn>((uint16_t)(e >> 16));
      if (x >= tau && x > kNegInf) {  // the fill of a ragged last granule is never a token
        ++f.n;
        if ((e & 0xffffu) != pos_a) fix_add(f, ex2((x - m) * kLog2e));
      }
    }
  } else {
    const int n_full = V / kElems, n_gran = (V + kElems - 1) / kElems;
    for (int g = tid; g < n_gran; g += nt) {
      Granule<TIn> gr;
      gr.load_any(row, V, n_full, g);
      float x[kElems];
      gr.get(x);
      const int ja = a - g * kElems;
#pragma unroll
      for (int j = 0; j < kElems; ++j) {
        if (x[j] >= tau && x[j] > kNegInf) {
          ++f.n;
          if (j != ja) fix_add(f, ex2((x[j] - m) * kLog2e));
        }
      }
    }
  }
  return f;
}

// Statistics of one side of one row.  `run` holds the start of the running bound (from an
// element of this row, or -inf) and is visible to the block.  When `next_row` is given,
// thread 0 leaves in `run_next` a start for that row: from the larger of its sampled
// token's logit and its granule at the position of this row's maximum.
template <typename TIn>
__device__ __forceinline__ SideStats side_stats_cs(const TIn *row, const TIn *next_row, int V, int n_steps,
                                                   int a, const RowParams &p, float log_rho_dn, WarpCand &wc,
                                                   unsigned long long *run, unsigned long long *run_next,
                                                   float *scratch, uint32_t *mask_row) {
  constexpr int kElems = Granule<TIn>::kElems;
  const bool has_a = a >= 0;
  const float z_a = has_a ? Storage<TIn>::widen(row[a]) : 0.f;
  wc.cnt = 0;
  wc.staged = 0;
  wc.tb_tried = kNegInf;
  const LogSum all = sweep1_cs<TIn>(row, V, n_steps, wc, run, log_rho_dn, scratch);

  float next_start = kNegInf;
  uint32_t next_g = 0xffffffffu;
  if (next_row && threadIdx.x == 0) {
    next_g = (uint32_t)*reinterpret_cast<volatile unsigned long long *>(run);
    if (has_a) next_start = Storage<TIn>::widen(next_row[a]);
    if (next_g != 0xffffffffu) {
      Granule<TIn> gr;
      gr.load_any(next_row, V, V / kElems, (int)next_g);
      next_start = fmaxf(next_start, gr.max());
    }
  }

  SideStats st;
  st.m = all.m;
  st.lse = lse_from_logsum(all);
  st.sum_c = (double)all.c;
  st.sum_s = all.s;
  st.tau = threshold_of<TIn>(all.m, p.log_rho, p.mode);
  st.z_a = z_a;
  st.member = has_a && z_a >= st.tau;
  st.e_a = st.member ? ex2((z_a - st.m) * kLog2e) : 0.f;

  const FixSum f = walk_sum<TIn>(row, V, n_steps, a, st.tau, st.m, wc);
  if (next_row && threadIdx.x == 0)
    *run_next = ((unsigned long long)float_key(Storage<TIn>::widen(Below<TIn>::of(
                     __fadd_rd(next_start, log_rho_dn)))) << 32) | next_g;
  const FixSum tot = block_reduce_fix(f, scratch);
  st.s_x = fix_value(tot);
  st.n = tot.n;
  set_mask_mass(st, V, p.mode, Storage<TIn>::widen(Storage<TIn>::narrow(p.mask_value)), has_a);

  if (mask_row) {  // optional packed membership mask (diagnostic output, plain loads)
    const int n_words = (V + 31) / 32;
    for (int w = threadIdx.x; w < n_words; w += blockDim.x) {
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

// Gradient row (Prop. 5.4, set fixed): a row of zeros, then the safe entries of each warp's
// list scattered into it.  A warp without a list sweeps its share of the row once more.
template <typename TIn, typename TGrad>
__device__ __forceinline__ void grad_cs(const TIn *row, TGrad *grow, int V, int a, const SideStats &st,
                                        float g, const WarpCand &wc) {
  constexpr int kElems = Granule<TIn>::kElems;
  const int nt = blockDim.x, tid = threadIdx.x, lane = tid & 31, wbase = tid & ~31;
  const int n_full = V / kElems;
  const int n_gran = (V + kElems - 1) / kElems;
  const float s_tot = st.s_x + st.e_a + st.s_mask;
  const bool live = st.live;
  const float coef = live ? -g / s_tot : 0.f;
  const float g_a = st.member ? g * ((st.s_x + st.s_mask) / s_tot) : 0.f;
  const int a_live = (live && st.member) ? a : -1;
  const float tau = st.tau, m = st.m;
  if (live && wc.cnt < 0) {
    for (int gi = tid; gi < n_gran; gi += nt) {
      Granule<TIn> gr;
      gr.load_any(row, V, n_full, gi);
      granule_grad<TIn, TGrad>(gr, grow, V, n_full, gi, a_live, tau, m, coef, g_a);
    }
    return;
  }
  for (int gi = tid; gi < n_gran; gi += nt) {
    if (gi < n_full) {
      if (DVP_IN((long long)gi * kElems + kElems - 1, V, DVP_OOB_GLOBAL))
        store_zero_granule<TGrad, kElems>(grow + (size_t)gi * kElems);
    } else {
      for (int j = 0; j < kElems; ++j) {
        const long long e = (long long)gi * kElems + j;
        if (e < V) grow[e] = Storage<TGrad>::narrow(0.f);
      }
    }
  }
  if (!live) return;
  __syncwarp();  // the zeros of this warp's granules are ordered before the entries written over them
  const uint32_t pos_a = (uint32_t)position_in_warp(a_live, kElems);
  for (int i = lane; i < wc.cnt; i += 32) {
    const uint32_t e = wc.list[i];
    const float x = widen_bits<TIn>((uint16_t)(e >> 16));
    if (!(x >= tau && x > kNegInf)) continue;
    const uint32_t pos = e & 0xffffu, ord = pos / kElems;
    const long long k = ((long long)(ord >> 5) * nt + wbase + (ord & 31u)) * kElems + pos % kElems;
    const float o = pos == pos_a ? g_a : coef * ex2((x - m) * kLog2e);
    if (DVP_IN(k, V, DVP_OOB_GLOBAL)) grow[k] = Storage<TGrad>::narrow(o);
  }
}

// Shared memory, in bytes: block reductions (160 words), the two running-bound words, the
// rings, the lists (cap entries per warp).
__host__ __device__ inline size_t smem_bytes_cs(int threads, int cap) {
  return 160 * 4 + 16 + (size_t)(threads / 32) * kRingBytes + (size_t)(threads / 32) * cap * 4;
}

// One block per token row; the two rows of a token (training, inference) are two passes of
// one loop body.  kWeighted: the upstream gradient is multiplied by the token's importance
// weight, which needs the inference side first: that instantiation takes the inference
// row in the first pass.
template <typename TIn, typename TGrad, int kThreads, int kBlocks, bool kWeighted>
__global__ void __launch_bounds__(kThreads, kBlocks) dvp_row_kernel_cs(const RowParams p, int n_steps, int cap) {
  extern __shared__ __align__(16) float smem[];
  float *scratch = smem;  // 160 words for the block reductions
  unsigned long long *run = reinterpret_cast<unsigned long long *>(smem + 160);
  const int warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  WarpCand wc;
  wc.ring = reinterpret_cast<uint4 *>(reinterpret_cast<char *>(smem + 164) + warp * kRingBytes);
  wc.list = reinterpret_cast<uint32_t *>(reinterpret_cast<char *>(smem + 164) + nwarp * kRingBytes) + warp * cap;
  wc.cap = cap;

  constexpr int kElems = Granule<TIn>::kElems;
  DVP_BOUNDS_BEGIN(p.bounds_status);
  DVP_BOUNDS_SET(n_gran, (p.V + kElems - 1) / kElems);
  DVP_BOUNDS_SET(V, p.V);
  DVP_BOUNDS_SET(n_ring, kRing);
  DVP_BOUNDS_SET(n_list, cap);
  DVP_BOUNDS_SYNC();
  const long long t = blockIdx.x;
  const long long id = p.ids ? load_id(p.ids, p.id_is_i32, t) : -1;
  const bool has_id = id >= 0, bad_id = id >= p.V;
  const int a = (has_id && !bad_id) ? (int)id : -1;
  const int V = (int)p.V;
  const TIn *trow = reinterpret_cast<const TIn *>(p.train) + t * p.ld_train;
  const TIn *irow = p.infer ? reinterpret_cast<const TIn *>(p.infer) + t * p.ld_infer : nullptr;

  // ln rho rounded down; with the threshold formed in the logits' type also its rounded form
  float log_rho_dn = __double2float_rd(p.log_rho);
  if (p.mode & DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE)
    log_rho_dn = fminf(log_rho_dn, Storage<TIn>::widen(Storage<TIn>::narrow((float)p.log_rho)));

  const bool infer_first = kWeighted && irow;
  if (threadIdx.x == 0) {
    const TIn *first = infer_first ? irow : trow;
    const float start = a >= 0 ? Storage<TIn>::widen(first[a]) : kNegInf;
    run[0] = ((unsigned long long)float_key(Storage<TIn>::widen(Below<TIn>::of(__fadd_rd(start, log_rho_dn))))
              << 32) | (a >= 0 ? (uint32_t)(a / kElems) : 0xffffffffu);
  }
  __syncthreads();

  const float nan = __int_as_float(0x7fc00000);
  float lp_t = nan, lp_i = nan;  // ln pi^mp(a) of the two sides (thread 0: as written to the outputs)
  int mem_t = 0, mem_i = 0;
  const int n_pass = irow ? 2 : 1;
#pragma unroll 1
  for (int pass = 0; pass < n_pass; ++pass) {
    const bool is_train = (pass == 0) != infer_first;
    const TIn *row = is_train ? trow : irow;
    const TIn *next_row = pass + 1 < n_pass ? (is_train ? irow : trow) : nullptr;
    uint32_t *mask_all = is_train ? p.out_t.mask : p.out_i.mask;
    uint32_t *mask_row = mask_all ? mask_all + t * ((p.V + 31) / 32) : nullptr;
    const SideStats s = side_stats_cs<TIn>(row, next_row, V, n_steps, a, p, log_rho_dn, wc, run + pass,
                                           run + 1, scratch, mask_row);
    float lp = a >= 0 ? logp_mp_of(s) : nan;
    if (is_train && p.grad) {
      float g = p.upstream[t];
      if constexpr (kWeighted) {
        float w;
        if (a < 0) {
          w = nan;
        } else if (p.infer) {
          const float r = (p.mode & DVP_MODE_FINITE_MASK) ? lp - lp_i : log_ratio_of(s.member, mem_i, lp, lp_i);
          w = token_weight(r, p.weight_kind, p.weight_lo, p.weight_hi);
        } else {
          w = row_weight_given(p, s, t, true);
        }
        if (w == w) g *= w;
        if (p.weight_out && threadIdx.x == 0) p.weight_out[t] = w;
      }
      grad_cs<TIn, TGrad>(trow, reinterpret_cast<TGrad *>(p.grad) + t * p.ld_grad, V, a, s, g, wc);
    }
    if (threadIdx.x == 0) {
      dvp_side_out o;
      o.max = is_train ? p.out_t.max : p.out_i.max;
      o.lse = is_train ? p.out_t.lse : p.out_i.lse;
      o.lse_safe = is_train ? p.out_t.lse_safe : p.out_i.lse_safe;
      o.logp = is_train ? p.out_t.logp : p.out_i.logp;
      o.logp_mp = is_train ? p.out_t.logp_mp : p.out_i.logp_mp;
      o.comp_mp = is_train ? p.out_t.comp_mp : p.out_i.comp_mp;
      o.count = is_train ? p.out_t.count : p.out_i.count;
      o.log_cov = is_train ? p.out_t.log_cov : p.out_i.log_cov;
      o.mask = nullptr;
      lp = finish_side(o, t, s, has_id, bad_id);
    }
    if (is_train) {
      lp_t = lp;
      mem_t = s.member;
    } else {
      lp_i = lp;
      mem_i = s.member;
    }
  }

  if (threadIdx.x == 0) {
    uint8_t flags = (uint8_t)((mem_t ? DVP_FLAG_IN_TRAIN : 0) | (has_id ? 0 : DVP_FLAG_NO_ID) |
                              (bad_id ? DVP_FLAG_BAD_ID : 0));
    if (p.infer) {
      if (mem_i) flags |= DVP_FLAG_IN_INFER;
      if (p.log_ratio)
        p.log_ratio[t] = !(has_id && !bad_id)              ? nan
                         : (p.mode & DVP_MODE_FINITE_MASK) ? lp_t - lp_i
                                                           : log_ratio_of(mem_t, mem_i, lp_t, lp_i);
    }
    if (p.flags) p.flags[t] = flags;
  }
}

}  // namespace cs
}  // namespace dvp
