// The row pass of the fused LM-head entry point over one panel of fp32 logits, with the
// normalisation deferred.
//
// The logits contraction leaves every row's maximum (in pieces), so the threshold of
// Def. 5.1 is known before the panel is read and one sweep gives everything: the full sum,
// the masked sum and the count (Def. 5.2), and, written as it goes, the panel
//     P_tk = 2^14 e^{z_tk - m_t}  for k in V_S, k != a_t;   0 otherwise          (float16)
// which is the gradient of Prop. 5.4 up to a factor per row that is known only at the end of
// the row: G_tk = c_t P_tk + 1[k = a_t] q_t with
//     c_t = -g_t / (2^14 s_S,t),   q_t = g_t s_{S\a},t / s_S,t   (= g_t (1 - pi^mp(a_t)), no cancellation).
// The factor goes where it costs nothing: d_hidden_t = c_t (P W)_t + q_t W_a (a row scale in the
// contraction's epilogue, one row of W added), d_w = P^T diag(c) hidden + sum_t q_t e_a hidden_t^T
// (the hidden rows are scaled while they are converted to float16, the 1[k = a] terms are
// added to d_w in a fixed order).  The panel is read once and written once.
#pragma once

#include "dvp_rows_impl.cuh"

namespace dvp {
namespace panel {

constexpr float kPScale = 16384.f;  // 2^14: P uses float16's normal range for members down to 4e-9 of the maximum

struct PanelParams {
  RowParams row;       // train = the fp32 panel; ids, upstream, T, V, ld_train, log_rho, outputs, weights
  const float *row_max;  // the row maxima that the logits contraction left, in pieces: the maximum of row t is
  long long row_max_ld;  // the largest of row_max[t * row_max_ld + i], i < row_max_n
  int row_max_n;
  __half *P;           // [T, ld_p]
  long long ld_p;
  float *row_scale;    // [T] c_t (0 for a row without a gradient): scale of the row in d_hidden's epilogue
  float *hid_scale;    // [T] c_t K, K = 2^14 * scale / 512: scale of the hidden row in d_w's contraction
                       // (|c_t K| < 32, so hidden entries up to 2047 fit float16)
  float *a_coef;       // [T] q_t (0 for a row without a gradient)
  const float *scale;  // device scalar, the power of two taken from max |upstream|
};

struct PanelSums {
  float s_all, s_safe_x;  // sums of e^{z - m}: every token; the safe set without the sampled token
  int n;                  // |V_S|
};

__device__ __forceinline__ void absorb_panel(const Granule<float> &gr, int g, int n_full, int V, int a, float m,
                                             float tau, PanelSums &acc, __half *prow) {
  constexpr int kElems = 8;
  float x[kElems];
  gr.get(x);
  const int ja = a - g * kElems;
  float all = 0.f;
  uint32_t w[4];
#pragma unroll
  for (int j = 0; j < kElems; j += 2) {
    float o[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const float e = ex2((x[j + u] - m) * kLog2e);  // the fill of a ragged last granule is -inf: e = 0
      all += e;
      const bool keep = x[j + u] >= tau && x[j + u] > kNegInf;
      o[u] = 0.f;
      if (keep) {
        ++acc.n;
        if (j + u != ja) {
          acc.s_safe_x += e;
          o[u] = e * kPScale;
        }
      }
    }
    const __half2 h2 = __floats2half2_rn(o[0], o[1]);
    w[j / 2] = *reinterpret_cast<const uint32_t *>(&h2);
  }
  acc.s_all += all;
  if (g < n_full) {
    st_stream16(prow + (size_t)g * kElems, make_uint4(w[0], w[1], w[2], w[3]));
  } else {
    const __half *h = reinterpret_cast<const __half *>(w);
#pragma unroll
    for (int j = 0; j < kElems; ++j) {
      const long long k = (long long)g * kElems + j;
      if (k < V) prow[k] = h[j];
    }
  }
}

template <int kThreads, int kBlocks>
__global__ void __launch_bounds__(kThreads, kBlocks) dvp_panel_kernel(const PanelParams pp) {
  __shared__ float scratch[96];
  const RowParams &p = pp.row;
  constexpr int kElems = 8, kStage = 2;
  const long long t = blockIdx.x;
  DVP_BOUNDS_BEGIN(p.bounds_status);
  DVP_BOUNDS_SET(n_gran, (p.V + kElems - 1) / kElems);
  DVP_BOUNDS_SET(V, p.V);
  DVP_BOUNDS_SYNC();
  const long long id = load_id(p.ids, p.id_is_i32, t);
  const bool has_id = id >= 0, bad_id = id >= p.V;
  const int a = (has_id && !bad_id) ? (int)id : -1;
  const int V = (int)p.V;
  const float *row = reinterpret_cast<const float *>(p.train) + t * p.ld_train;
  __half *prow = pp.P + t * pp.ld_p;

  const float *pieces = pp.row_max + t * pp.row_max_ld;
  float mx = kNegInf;
  for (int i = threadIdx.x; i < pp.row_max_n; i += blockDim.x) mx = fmaxf(mx, pieces[i]);
  const float m = block_reduce_max(mx, scratch);

  SideStats st;
  st.m = m;
  st.tau = threshold_f32(m, p.log_rho);
  const bool has_a = a >= 0;
  st.z_a = has_a ? row[a] : 0.f;
  st.member = has_a && st.z_a >= st.tau;
  st.e_a = st.member ? ex2((st.z_a - m) * kLog2e) : 0.f;

  const int n_full = V / kElems;
  const int n_gran = (V + kElems - 1) / kElems;
  const int per_step = kStage * (int)blockDim.x;
  const int n_steps = (n_gran + per_step - 1) / per_step;
  PanelSums acc = {0.f, 0.f, 0};
  if (n_steps > 0) {  // two stages in flight, as in the row kernels
    Stage<float, kStage> s0, s1;
    s0.load(row, V, n_full, 0);
    int step = 0;
    for (; step + 1 < n_steps; step += 2) {
      s1.load(row, V, n_full, step + 1);
#pragma unroll
      for (int u = 0; u < kStage; ++u)
        absorb_panel(s0.g[u], (step * kStage + u) * (int)blockDim.x + (int)threadIdx.x, n_full, V, a, m, st.tau, acc,
                     prow);
      if (step + 2 < n_steps) s0.load(row, V, n_full, step + 2);
#pragma unroll
      for (int u = 0; u < kStage; ++u)
        absorb_panel(s1.g[u], ((step + 1) * kStage + u) * (int)blockDim.x + (int)threadIdx.x, n_full, V, a, m,
                     st.tau, acc, prow);
    }
    if (step < n_steps) {
#pragma unroll
      for (int u = 0; u < kStage; ++u)
        absorb_panel(s0.g[u], (step * kStage + u) * (int)blockDim.x + (int)threadIdx.x, n_full, V, a, m, st.tau, acc,
                     prow);
    }
  }
  const SumCount safe = block_reduce_sumcount({acc.s_safe_x, acc.n}, scratch);
  const SumCount all = block_reduce_sumcount({acc.s_all, 0}, scratch);
  st.s_x = safe.s;
  st.n = safe.n;
  st.lse = (double)m + (double)logf(all.s);
  st.sum_c = (double)m * (double)kLog2e;
  st.sum_s = all.s;
  set_mask_mass(st, V, 0, 0.f, has_a);

  if (threadIdx.x == 0) {
    finish_side(p.out_t, t, st, has_id, bad_id);
    if (p.flags)
      p.flags[t] = (uint8_t)((st.member ? DVP_FLAG_IN_TRAIN : 0) | (has_id ? 0 : DVP_FLAG_NO_ID) |
                             (bad_id ? DVP_FLAG_BAD_ID : 0));
    float g = p.upstream[t];
    if (p.weight_kind != DVP_WEIGHT_NONE) {
      const float w = row_weight_given(p, st, t, a >= 0);
      if (w == w) g *= w;
      if (p.weight_out) p.weight_out[t] = w;
    }
    // a missing sampled token, or a pruned one, has weight zero: no gradient from this row
    const bool live = st.live && st.member;
    const float s_safe = st.s_x + st.e_a;  // >= 1: the maximum is always in the set
    const float c = live ? -g / (s_safe * kPScale) : 0.f;
    pp.row_scale[t] = c;
    pp.hid_scale[t] = live ? -g * (*pp.scale * (1.f / 512.f)) / s_safe : 0.f;
    pp.a_coef[t] = live ? g * (st.s_x / s_safe) : 0.f;
  }
  if (p.out_t.mask) {  // optional packed membership mask (diagnostic output, plain loads)
    uint32_t *mask_row = p.out_t.mask + t * ((p.V + 31) / 32);
    const int n_words = (V + 31) / 32;
    for (int w = threadIdx.x; w < n_words; w += blockDim.x) {
      uint32_t bits = 0;
      for (int b = 0; b < 32; ++b) {
        const long long k = (long long)w * 32 + b;
        if (k < V && row[k] >= st.tau) bits |= 1u << b;
      }
      mask_row[w] = bits;
    }
  }
}

// d_hidden[t, :] += q_t W[a_t, :]: the 1[k = a] term of the gradient row, in fp32.
__global__ void __launch_bounds__(256) add_sampled_rows_kernel(float *d_hidden, long long ld_dh,
                                                               const __nv_bfloat16 *w, long long ld_w,
                                                               const void *ids, int id_is_i32, const float *a_coef,
                                                               int H) {
  const long long t = blockIdx.x;
  const float q = a_coef[t];
  if (q == 0.f) return;
  const long long a = load_id(ids, id_is_i32, t);
  const __nv_bfloat16 *wa = w + a * ld_w;
  float *out = d_hidden + t * ld_dh;
  for (int h = threadIdx.x; h < H; h += blockDim.x) out[h] = fmaf(q, __bfloat162float(wa[h]), out[h]);
}

// The tokens of a chunk (at most 4096) whose row has a gradient, sorted by (sampled id, token):
// tokens that share a vocabulary row are then neighbours, in token order.  Keys: id << 12 | token;
// the others sort to the end as all ones.
constexpr int kSortChunk = 4096;
__global__ void __launch_bounds__(1024) sort_sampled_ids_kernel(const void *ids, int id_is_i32, const float *a_coef,
                                                                int rows, unsigned long long *sorted) {
  __shared__ unsigned long long key[kSortChunk];
  for (int i = threadIdx.x; i < kSortChunk; i += blockDim.x) {
    unsigned long long k = ~0ull;
    if (i < rows && a_coef[i] != 0.f) k = ((unsigned long long)load_id(ids, id_is_i32, i) << 12) | (unsigned)i;
    key[i] = k;
  }
  __syncthreads();
  for (int size = 2; size <= kSortChunk; size <<= 1) {  // bitonic network, ascending
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = threadIdx.x; i < kSortChunk / 2; i += blockDim.x) {
        const int lo = 2 * i - (i & (stride - 1)), hi = lo + stride;
        const bool up = (lo & size) == 0;
        const unsigned long long x = key[lo], y = key[hi];
        if ((x > y) == up) {
          key[lo] = y;
          key[hi] = x;
        }
      }
      __syncthreads();
    }
  }
  for (int i = threadIdx.x; i < kSortChunk; i += blockDim.x) sorted[i] = key[i];
}

// d_w[a, :] += sum over the tokens t of the chunk with a_t = a, in token order, of q_t hidden[t, :].
// One block per sorted position; the block at the head of a run of equal ids does the run.
__global__ void __launch_bounds__(256) add_sampled_hidden_kernel(const unsigned long long *sorted,
                                                                 const float *a_coef, const __nv_bfloat16 *hidden,
                                                                 long long ld_hidden, float *d_w, long long ld_dw,
                                                                 int H) {
  const int i = blockIdx.x;
  const unsigned long long k = sorted[i];
  if (k == ~0ull) return;
  const unsigned long long a = k >> 12;
  if (i > 0 && (sorted[i - 1] >> 12) == a) return;
  float *out = d_w + (long long)a * ld_dw;
  for (int h = threadIdx.x; h < H; h += blockDim.x) {
    float acc = 0.f;
    for (int j = i; j < kSortChunk; ++j) {
      const unsigned long long kj = sorted[j];
      if (kj == ~0ull || (kj >> 12) != a) break;
      const int t = (int)(kj & 4095u);
      acc = fmaf(a_coef[t], __bfloat162float(hidden[(long long)t * ld_hidden + h]), acc);
    }
    out[h] += acc;
  }
}

}  // namespace panel
}  // namespace dvp
