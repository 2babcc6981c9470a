// Tensor-core contraction C[M,N] (+)= alpha * A[M,K] * B[N,K]^T for sm_100a.
//
// A and B are 16-bit (both bf16 or both f16), row-major with K contiguous; C is
// fp32 row-major.  A persistent kernel, one block per SM, walks 128 x 256 output
// tiles.  Per tile the K dimension is cut in slices of 64: a producer thread
// brings the A (128 x 64) and B (256 x 64) slices into a ring of shared-memory
// stages with TMA tile loads (128-byte swizzle), one thread issues tcgen05.mma
// (M = 128, N = 256, K = 16, four per slice) accumulating in tensor memory, and
// four epilogue warps read the accumulator back with tcgen05.ld, scale it and
// store it.  Two accumulators (2 x 256 TMEM columns) let the epilogue of one
// tile overlap the MMAs of the next.
//
// Every wait on an mbarrier is bounded.  A wait that runs out records a code in
// *status, raises a block-wide abort flag, and every role leaves its loop; the
// block then lets its own copies land, frees its tensor memory and returns.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dvp {
namespace gemm {

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kStages = 4;
constexpr int kUmmaK = 16;
constexpr int kThreads = 192;  // warp 0: TMA, warp 1: MMA, warps 2..5: epilogue
constexpr uint32_t kBytesA = kBM * kBK * 2, kBytesB = kBN * kBK * 2;
constexpr uint32_t kStageBytes = kBytesA + kBytesB;
constexpr uint32_t kTmemCols = 512;
constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + 256;
constexpr uint32_t kSpinLimit = 1u << 22;

enum { kErrNone = 0, kErrProducerWait = 11, kErrMmaWaitFull = 12, kErrMmaWaitTmem = 13,
       kErrEpilogueWait = 14 };

struct Params {
  float *C;
  long long ldc;
  int M, N, K;
  float alpha;
  const float *alpha_dev;  // optional device scalar multiplied into alpha
  int accumulate;          // C += instead of C =
  int *status;             // device word, set non-zero when a wait gives up
  int a_mn_major;          // A is stored transposed, [K, M] with M contiguous (pair kernel only)
  int split_k;             // pair kernel: each tile's K range is cut into this many units whose
                           // results are added to C with atomics (C zeroed or accumulated into)
  float *row_max;          // optional (pair kernel, no split, no accumulation): row_max[row * row_max_ld + tn]
  long long row_max_ld;    // = the maximum of row `row` of C over the columns of tile column tn
  const float *row_scale;  // optional (pair kernel): row `row` of the product is multiplied by row_scale[row]
};

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
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit ran out or another role raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 32) __nanosleep(40);
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x,
                                            int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
      "%4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of
// 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);  // start address
  d |= (uint64_t)1 << 16;                   // leading byte offset (unused with swizzle): 16 B
  d |= (uint64_t)(1024 >> 4) << 32;         // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                   // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                   // 128-byte swizzle
  return d;
}

// The same for an MN-major operand (stored [K, MN] with MN contiguous), brought in as
// boxes of 64 K-rows x 64 MN-elements: inside a box a K-row is 128 swizzled bytes, groups
// of 8 K-rows are 1024 bytes apart (stride byte offset), and the next 64 MN-elements
// start one box (8192 bytes) further (leading byte offset).
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);
  d |= (uint64_t)(8192 >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor for kind::f16: fp32 accumulate, A and B of format
// `fmt` (0 = f16, 1 = bf16), both K-major, M = 128, N = 256.
__device__ __forceinline__ uint32_t instr_desc(uint32_t fmt) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kBN >> 3) << 17) |
         ((uint32_t)(kBM >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                     uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

struct Shared {
  uint64_t full[kStages], empty[kStages], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
gemm_tn_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const Params p, const uint32_t fmt) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms are 1024-byte aligned
  uint8_t *aligned = smem_raw + (base - smem_u32(smem_raw));
  Shared *sh = reinterpret_cast<Shared *>(aligned + (size_t)kStages * kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const int tiles_m = (p.M + kBM - 1) / kBM, tiles_n = (p.N + kBN - 1) / kBN;
  const int n_tiles = tiles_m * tiles_n;
  const int k_slices = (p.K + kBK - 1) / kBK;
  // Blocks that run together take consecutive tiles: walk the shorter tile dimension
  // fastest so that they share the operand panel of the longer one through L2.
  const bool m_fastest = tiles_m <= tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh->tmem_full[b]), 1);
      mbar_init(smem_u32(&sh->tmem_empty[b]), 4);
    }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // one warp allocates the tensor memory of the block
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sh->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  volatile int *abort_flag = &sh->abort_flag;

  if (warp == 0) {
    // ---------------- producer: TMA loads into the stage ring
    if (lane == 0) {
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x) {
        const int tm = m_fastest ? tile % tiles_m : tile / tiles_n;
        const int tn = m_fastest ? tile / tiles_m : tile % tiles_n;
        for (int ks = 0; ks < k_slices; ++ks, ++it) {
          const uint32_t s = it % kStages, round = it / kStages;
          if (round > 0 && !mbar_wait(smem_u32(&sh->empty[s]), (round - 1) & 1, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrProducerWait); }
            break;
          }
          const uint32_t bar = smem_u32(&sh->full[s]);
          mbar_expect_tx(bar, kStageBytes);
          const uint32_t dst = base + s * kStageBytes;
          tma_load_2d(dst, &map_a, bar, ks * kBK, tm * kBM);
          tma_load_2d(dst + kBytesA, &map_b, bar, ks * kBK, tn * kBN);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc(fmt);
      uint32_t it = 0, local_tile = 0;
      for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x, ++local_tile) {
        const uint32_t buf = local_tile & 1, use = local_tile >> 1;
        if (use > 0 && !mbar_wait(smem_u32(&sh->tmem_empty[buf]), (use - 1) & 1, abort_flag)) {
          if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrMmaWaitTmem); }
          break;
        }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * kBN;
        bool ok = true;
        for (int ks = 0; ks < k_slices; ++ks, ++it) {
          const uint32_t s = it % kStages, round = it / kStages;
          if (!mbar_wait(smem_u32(&sh->full[s]), round & 1, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrMmaWaitFull); }
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = base + s * kStageBytes, b_addr = a_addr + kBytesA;
          const uint64_t adesc = smem_desc_sw128(a_addr), bdesc = smem_desc_sw128(b_addr);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            // 16 elements of K are 32 bytes inside the 128-byte swizzled row
            const uint64_t step = (uint64_t)((k * kUmmaK * 2) >> 4);
            umma(tmem_d, adesc + step, bdesc + step, idesc, (ks > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&sh->empty[s]));  // the stage is free once these MMAs have read it
        }
        if (!ok) break;
        umma_commit(smem_u32(&sh->tmem_full[buf]));  // accumulator complete
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> global
    const int quarter = warp & 3;  // TMEM lanes this warp may read
    const float alpha = p.alpha * (p.alpha_dev ? *p.alpha_dev : 1.f);
    uint32_t local_tile = 0;
    for (int tile = blockIdx.x; tile < n_tiles && !*abort_flag; tile += gridDim.x, ++local_tile) {
      const int tm = m_fastest ? tile % tiles_m : tile / tiles_n;
      const int tn = m_fastest ? tile / tiles_m : tile % tiles_n;
      const uint32_t buf = local_tile & 1, use = local_tile >> 1;
      if (!mbar_wait(smem_u32(&sh->tmem_full[buf]), use & 1, abort_flag)) {
        if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrEpilogueWait); }
        break;
      }
      tc_fence_after();
      const int row = tm * kBM + quarter * 32 + lane;
      float *crow = p.C + (long long)row * p.ldc;
#pragma unroll 1
      for (int c0 = 0; c0 < kBN; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kBN + c0, r);
        tmem_wait_ld();
        const int col = tn * kBN + c0;
        if (row < p.M && col < p.N) {
          if (col + 32 <= p.N) {
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint32_t w[8];
              if (p.accumulate) {
                const float4 o0 = *reinterpret_cast<const float4 *>(crow + col + j);
                const float4 o1 = *reinterpret_cast<const float4 *>(crow + col + j + 4);
                const float old[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e)
                  w[e] = __float_as_uint(fmaf(alpha, __uint_as_float(r[j + e]), old[e]));
              } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) w[e] = __float_as_uint(alpha * __uint_as_float(r[j + e]));
              }
              asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(crow + col + j),
                           "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]),
                           "r"(w[7])
                           : "memory");
            }
          } else {
            for (int j = 0; j < 32 && col + j < p.N; ++j) {
              const float v = alpha * __uint_as_float(r[j]);
              crow[col + j] = p.accumulate ? crow[col + j] + v : v;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[buf]));
    }
  }

  // ---------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    // give this block's copies in flight time to land before the memory is released
    for (int i = 0; i < 2000; ++i) __nanosleep(500);
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols)
                 : "memory");
  }
}

// ---- the same contraction on pairs of blocks (tcgen05 cta_group::2) ------------------
// Two blocks of a cluster share one 256 x 256 output tile: each holds 128 rows of
// A, 128 of the 256 rows of B, and the 128 x 256 accumulator of its own rows in its
// tensor memory.  One thread of the leader block (cluster rank 0) issues the MMAs for
// both, so each block reads only half of B from shared memory per MMA: this removes
// the shared-memory bandwidth ceiling of the one-block form.  Both blocks' TMA loads
// complete on the leader's "full" barrier; the MMA thread's commits arrive on the
// "empty" and "accumulator full" barriers of both blocks; both blocks' epilogue warps
// arrive on the leader's "accumulator empty" barrier.

constexpr int kPairBM = 256;
constexpr int kStages2 = 6;
constexpr uint32_t kBytesB2 = (kBN / 2) * kBK * 2;
constexpr uint32_t kStageBytes2 = kBytesA + kBytesB2;
constexpr size_t kSmemBytes2 = 1024 + (size_t)kStages2 * kStageBytes2 + 256;

struct Shared2 {
  uint64_t full[kStages2], empty[kStages2], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of this block's shared-memory location `local` as seen in block `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr)
               : "memory");
}
// TMA tile load whose completion is counted on a barrier that may live in the peer block.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map,
                                                 uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], "
      "[%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void umma_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive, once these MMAs are done, on the barrier at this offset in both blocks of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], "
      "%1;" ::"r"(bar),
      "h"(mask)
      : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_tn_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const Params p, const uint32_t fmt) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *aligned = smem_raw + (base - smem_u32(smem_raw));
  Shared2 *sh = reinterpret_cast<Shared2 *>(aligned + (size_t)kStages2 * kStageBytes2);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  const int tiles_m = (p.M + kPairBM - 1) / kPairBM, tiles_n = (p.N + kBN - 1) / kBN;
  const int n_tiles = tiles_m * tiles_n;
  const int k_slices = (p.K + kBK - 1) / kBK;
  const bool m_fastest = tiles_m <= tiles_n;
  // work units: every tile once per K range; unit u is tile u % n_tiles of range u / n_tiles
  const int n_units = n_tiles * p.split_k;
  const int k_per = (k_slices + p.split_k - 1) / p.split_k;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages2; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);   // the leader's producer, plus the bytes of both blocks
      mbar_init(smem_u32(&sh->empty[s]), 1);  // one commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh->tmem_full[b]), 1);   // one commit
      mbar_init(smem_u32(&sh->tmem_empty[b]), 8);  // four epilogue warps in each block
    }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sh->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_barrier();  // barriers of both blocks are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  volatile int *abort_flag = &sh->abort_flag;

  if (warp == 0) {
    // ---------------- producer (both blocks): own rows of A, own half of B
    if (lane == 0) {
      uint32_t it = 0;
      for (int unit = pair; unit < n_units && !*abort_flag; unit += n_pairs) {
        const int tile = unit % n_tiles, k_lo = (unit / n_tiles) * k_per;
        const int k_hi = min(k_slices, k_lo + k_per);
        const int tm = m_fastest ? tile % tiles_m : tile / tiles_n;
        const int tn = m_fastest ? tile / tiles_m : tile % tiles_n;
        for (int ks = k_lo; ks < k_hi; ++ks, ++it) {
          const uint32_t s = it % kStages2, round = it / kStages2;
          if (round > 0 && !mbar_wait(smem_u32(&sh->empty[s]), (round - 1) & 1, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrProducerWait); }
            break;
          }
          const uint32_t bar_local = smem_u32(&sh->full[s]);
          if (rank == 0) mbar_expect_tx(bar_local, 2 * kStageBytes2);
          const uint32_t bar = map_to_rank(bar_local, 0);
          const uint32_t dst = base + s * kStageBytes2;
          if (p.a_mn_major) {  // two boxes of 64 K-rows x 64 rows of A
            const int m0 = tm * kPairBM + (int)rank * kBM;
            tma_load_2d_pair(dst, &map_a, bar, m0, ks * kBK);
            tma_load_2d_pair(dst + kBytesA / 2, &map_a, bar, m0 + 64, ks * kBK);
          } else {
            tma_load_2d_pair(dst, &map_a, bar, ks * kBK, tm * kPairBM + (int)rank * kBM);
          }
          tma_load_2d_pair(dst + kBytesA, &map_b, bar, ks * kBK, tn * kBN + (int)rank * (kBN / 2));
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader block only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kBN >> 3) << 17) |
                             ((uint32_t)(kPairBM >> 4) << 24) | (p.a_mn_major ? (1u << 15) : 0u);
      // bytes between two K = 16 steps of A: 32 inside a K-major row, 16 K-rows of an MN-major box
      const uint32_t a_step_bytes = p.a_mn_major ? 16u * 128u : (uint32_t)(kUmmaK * 2);
      uint32_t it = 0, local_tile = 0;
      for (int unit = pair; unit < n_units && !*abort_flag; unit += n_pairs, ++local_tile) {
        const int k_lo = (unit / n_tiles) * k_per, k_hi = min(k_slices, k_lo + k_per);
        const uint32_t buf = local_tile & 1, use = local_tile >> 1;
        if (use > 0 && !mbar_wait(smem_u32(&sh->tmem_empty[buf]), (use - 1) & 1, abort_flag)) {
          if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrMmaWaitTmem); }
          break;
        }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * kBN;
        bool ok = true;
        for (int ks = k_lo; ks < k_hi; ++ks, ++it) {
          const uint32_t s = it % kStages2, round = it / kStages2;
          if (!mbar_wait(smem_u32(&sh->full[s]), round & 1, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrMmaWaitFull); }
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = base + s * kStageBytes2, b_addr = a_addr + kBytesA;
          const uint64_t adesc = p.a_mn_major ? smem_desc_sw128_mn(a_addr) : smem_desc_sw128(a_addr);
          const uint64_t bdesc = smem_desc_sw128(b_addr);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            const uint64_t step = (uint64_t)((k * kUmmaK * 2) >> 4);
            const uint64_t a_step = (uint64_t)((k * a_step_bytes) >> 4);
            umma_pair(tmem_d, adesc + a_step, bdesc + step, idesc, (ks > k_lo || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(smem_u32(&sh->empty[s]));
        }
        if (!ok) break;
        umma_commit_pair(smem_u32(&sh->tmem_full[buf]));
      }
    }
  } else {
    // ---------------- epilogue (both blocks): own 128 rows of the pair's tile
    const int quarter = warp & 3;
    const float alpha_all = p.alpha * (p.alpha_dev ? *p.alpha_dev : 1.f);
    uint32_t local_tile = 0;
    for (int unit = pair; unit < n_units && !*abort_flag; unit += n_pairs, ++local_tile) {
      const int tile = unit % n_tiles;
      const int tm = m_fastest ? tile % tiles_m : tile / tiles_n;
      const int tn = m_fastest ? tile / tiles_m : tile % tiles_n;
      const uint32_t buf = local_tile & 1, use = local_tile >> 1;
      if (!mbar_wait(smem_u32(&sh->tmem_full[buf]), use & 1, abort_flag)) {
        if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, kErrEpilogueWait); }
        break;
      }
      tc_fence_after();
      const int row = tm * kPairBM + (int)rank * kBM + quarter * 32 + lane;
      float *crow = p.C + (long long)row * p.ldc;
      const float alpha = alpha_all * ((p.row_scale && row < p.M) ? p.row_scale[row] : 1.f);
      float row_hi = -__builtin_huge_valf();  // maximum of what this thread stores of its row
#pragma unroll 1
      for (int c0 = 0; c0 < kBN; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kBN + c0, r);
        tmem_wait_ld();
        const int col = tn * kBN + c0;
        if (p.row_max && row < p.M) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (col + j < p.N) row_hi = fmaxf(row_hi, alpha * __uint_as_float(r[j]));
        }
        if (row < p.M && col < p.N) {
          if (p.split_k > 1) {  // this unit holds a part of the sum: add it
            for (int j = 0; j < 32 && col + j < p.N; ++j) atomicAdd(crow + col + j, alpha * __uint_as_float(r[j]));
          } else if (col + 32 <= p.N) {
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint32_t w[8];
              if (p.accumulate) {
                const float4 o0 = *reinterpret_cast<const float4 *>(crow + col + j);
                const float4 o1 = *reinterpret_cast<const float4 *>(crow + col + j + 4);
                const float old[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e)
                  w[e] = __float_as_uint(fmaf(alpha, __uint_as_float(r[j + e]), old[e]));
              } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) w[e] = __float_as_uint(alpha * __uint_as_float(r[j + e]));
              }
              asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(crow + col + j),
                           "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]),
                           "r"(w[7])
                           : "memory");
            }
          } else {
            for (int j = 0; j < 32 && col + j < p.N; ++j) {
              const float v = alpha * __uint_as_float(r[j]);
              crow[col + j] = p.accumulate ? crow[col + j] + v : v;
            }
          }
        }
      }
      if (p.row_max && row < p.M) p.row_max[(long long)row * p.row_max_ld + tn] = row_hi;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(map_to_rank(smem_u32(&sh->tmem_empty[buf]), 0));
    }
  }

  // ---------------- teardown: nobody frees tensor memory the pair still uses
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    for (int i = 0; i < 2000; ++i) __nanosleep(500);
  }
  cluster_barrier();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols)
                 : "memory");
  }
}

// ---- host side ------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// Tensor map of a row-major [rows, k] 16-bit matrix (row stride ld elements)
// for boxes of box_rows x 64 with the 128-byte swizzle; reads past the extents
// return zeros.
inline bool make_map(CUtensorMap *map, const void *base, long long rows, long long k, long long ld,
                     int box_rows, bool is_bf16) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)k, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
            const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// C[M,N] (+)= alpha * A[M,K] * B[N,K]^T.  lda, ldb multiples of 8; ldc of 8; bases 16-byte
// (A, B) and 32-byte (C) aligned.  Returns a CUDA error code; cudaErrorInvalidValue for
// layouts it cannot take.
inline cudaError_t launch_gemm_tn(const void *A, long long lda, const void *B, long long ldb, float *C,
                                  long long ldc, int M, int N, int K, bool is_bf16, float alpha,
                                  const float *alpha_dev, bool accumulate, int *status, int sm_count,
                                  cudaStream_t stream, bool single_block_tiles = false,
                                  bool a_mn_major = false, int split_k = 1, float *row_max = nullptr,
                                  long long row_max_ld = 0, const float *row_scale = nullptr) {
  if (M <= 0 || N <= 0 || K <= 0) return cudaSuccess;
  if (lda % 8 || ldb % 8 || ldc % 8 || (uintptr_t)A % 16 || (uintptr_t)B % 16 || (uintptr_t)C % 32)
    return cudaErrorInvalidValue;
  if (a_mn_major && single_block_tiles) return cudaErrorInvalidValue;
  // every K range of a split needs work; the split results meet in C by atomic adds
  if (single_block_tiles || split_k < 1 || (K + kBK - 1) / kBK < 2 * split_k) split_k = 1;
  // per-tile row maxima are those of the stored values: only where a tile is stored once, whole
  if (row_max && (single_block_tiles || split_k > 1 || accumulate)) return cudaErrorInvalidValue;
  if (row_scale && single_block_tiles) return cudaErrorInvalidValue;
  Params p{C, ldc, M, N, K, alpha, alpha_dev, accumulate ? 1 : 0, status, a_mn_major ? 1 : 0, split_k,
           row_max, row_max_ld, row_scale};
  if (split_k > 1 && !accumulate) {
    const cudaError_t z = cudaMemset2DAsync(C, (size_t)ldc * 4, 0, (size_t)N * 4, (size_t)M, stream);
    if (z != cudaSuccess) return z;
  }
  CUtensorMap map_a, map_b;
  if (!single_block_tiles) {
    // pairs of blocks on 256 x 256 tiles; a transposed A is [K, M]: its "rows" are K, boxes of 64 x 64
    const bool ok_a = a_mn_major ? make_map(&map_a, A, K, M, lda, 64, is_bf16)
                                 : make_map(&map_a, A, M, K, lda, kBM, is_bf16);
    if (!ok_a || !make_map(&map_b, B, N, K, ldb, kBN / 2, is_bf16)) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(gemm_tn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSmemBytes2);
    if (e != cudaSuccess) return e;
    const int tiles = ((M + kPairBM - 1) / kPairBM) * ((N + kBN - 1) / kBN) * split_k;
    int pairs = sm_count / 2;
    if (pairs > tiles) pairs = tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes2;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_tn_pair_kernel, map_a, map_b, p, is_bf16 ? 1u : 0u);
  }
  if (!make_map(&map_a, A, M, K, lda, kBM, is_bf16) || !make_map(&map_b, B, N, K, ldb, kBN, is_bf16))
    return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(gemm_tn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kSmemBytes);
  if (e != cudaSuccess) return e;
  const int tiles = ((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
  const int grid = tiles < sm_count ? tiles : sm_count;
  gemm_tn_kernel<<<grid, kThreads, kSmemBytes, stream>>>(map_a, map_b, p, is_bf16 ? 1u : 0u);
  return cudaGetLastError();
}

}  // namespace gemm
}  // namespace dvp
