/*
 * dvp.h -- C ABI of the B200 (sm_100a) Dynamic Vocabulary Pruning library.
 *
 * The library turns [T, V] logit matrices into the pruned objective of
 * "Dynamic Vocabulary Pruning: Stable LLM-RL by Taming the Tail"
 * (arXiv 2512.23087).  Per token row (one state s), with logits z, sampled
 * token a, threshold rho and L = ln(rho):
 *
 *   safe set      V_S = { k : z_k >= max_j z_j + L }        Def. 5.1, in the
 *                 logit-space form of App. A (protocol 2); equality is kept
 *   coverage      Z = sum_{k in V_S} pi(k)                   Def. 5.2
 *   pruned policy pi^mp(a) = pi(a) / Z on V_S, 0 elsewhere   Def. 5.2, Prop. 5.6(1)
 *   gradient      d log pi^mp(a) / d z_k = 1[k=a] - pi^mp(k) on V_S, 0 off it,
 *                 safe set held fixed                        Prop. 5.4, Prop. 5.6(2)
 *   log-ratio     ln pi^mp_train(a) - ln pi^mp_infer(a)      Thm. 4.1 (sign), Thm. 5.3,
 *                                                            App. A (protocol 4)
 *
 * Conventions that hold for every entry point
 *   - Every pointer marked "device" is a CUDA device pointer owned by the
 *     caller; the library never allocates, frees or retains it.
 *   - A call validates its arguments on the host, enqueues kernels on
 *     `stream` (a cudaStream_t passed as void*) and returns without
 *     synchronising.  Outputs are valid once the stream reaches that point.
 *   - Return value: a dvp_status.  Host-detectable problems are reported
 *     before anything is launched.  Problems only the device can see (a
 *     sampled id outside [0, V)) set DVP_FLAG_BAD_ID for that token, give it
 *     NaN log-probabilities and a zero gradient row; nothing traps.
 *   - Matrices are row-major with a row stride `ld*` counted in elements.
 *   - `struct_size` must equal sizeof of the struct the caller compiled with.
 *   - Logits must be finite.  Behaviour on NaN or infinite logits is
 *     unspecified (no fault, but the numbers mean nothing).
 *   - rho lies in [0, 1].  rho = 0 keeps every token (full log-softmax);
 *     rho = 1 keeps the argmax and its exact ties.
 *   - The membership test is exact: it equals the comparison of the stored
 *     logit, widened to double, against (double)max + log(rho) in double.
 */
#ifndef DVP_H_
#define DVP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DVP_OK = 0,
  DVP_ERR_INVALID_ARG = 1, /* null pointer, bad size, rho outside [0,1], ... */
  DVP_ERR_UNSUPPORTED = 2, /* dtype, device architecture or size not handled */
  DVP_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small     */
  DVP_ERR_CUDA = 4         /* a CUDA runtime call failed                     */
} dvp_status;

typedef enum { DVP_F32 = 0, DVP_BF16 = 1, DVP_F16 = 2 } dvp_dtype;
typedef enum { DVP_ID_I64 = 0, DVP_ID_I32 = 1 } dvp_id_dtype;

/* bits of the per-token flags byte */
enum {
  DVP_FLAG_IN_TRAIN = 1, /* a is in the training safe set V_S               */
  DVP_FLAG_IN_INFER = 2, /* a is in the inference safe set V'_S             */
  DVP_FLAG_NO_ID = 64,   /* id < 0: row statistics only                     */
  DVP_FLAG_BAD_ID = 128  /* id >= V                                         */
};

/*
 * bits of `mode` (dvp_forward_args, dvp_backward_args); 0 is the paper's definition.
 *   DVP_MODE_FINITE_MASK  pruned logits are replaced by the finite `mask_value`
 *       (rounded to the logits' type) and stay in the partition sum, as in the
 *       listing of App. A and Sec. 5.5 ("-50.0 in BF16"): lse_safe becomes the
 *       log-sum-exp of the masked row, logp_mp of a pruned sampled token is
 *       mask_value - lse_safe (finite), log_ratio is always finite, and a pruned
 *       sampled token still sends -g softmax(masked)_k to the kept positions.
 *       Assumes max logit >= mask_value - 80.
 *   DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE  the threshold is formed as an eager
 *       tensor expression of the logits' type forms it: log(rho) rounded to that
 *       type, added to the max in float32, the sum rounded to that type again.
 */
enum { DVP_MODE_FINITE_MASK = 1, DVP_MODE_THRESHOLD_IN_LOGITS_DTYPE = 2 };

enum { DVP_ENTRY_FORWARD = 0, DVP_ENTRY_BACKWARD = 1, DVP_ENTRY_FUSED_LMHEAD = 2 };

/*
 * `weight_kind` of dvp_forward_args: the per-token upstream gradient is
 * multiplied inside the kernel by a token-level importance weight w_t formed
 * from the token's own log-ratio r_t = ln pi^mp_train(a_t) - ln pi^mp_infer(a_t)
 * (the per-token factor of the estimator of Thm. 5.3, computed as the
 * exponential of a difference of log-probabilities, App. A protocol 4) and held
 * constant, so that one call gives the gradient of
 * sum_t upstream_t * stopgrad(w_t) * ln pi^mp_train(a_t):
 *   DVP_WEIGHT_NONE      w = 1 (upstream is used as given)
 *   DVP_WEIGHT_RATIO     w = e^r
 *   DVP_WEIGHT_TRUNCATE  w = min(e^r, weight_hi)      (truncated importance sampling)
 *   DVP_WEIGHT_MASK      w = e^r if weight_lo <= e^r <= weight_hi, else 0
 *                                                      (masked importance sampling)
 * r = -inf (a outside V_S) gives w = 0; r = +inf (a outside V'_S only) gives
 * +inf, weight_hi and 0.  Sec. 6 names the two comparison methods and "a
 * threshold of 0.2" without saying what it bounds: the bounds are the caller's.
 * Sequence-level weights (the product over a trajectory) and the token veto need
 * every token of the sequence first: use dvp_sequence_aggregate and dvp_backward.
 */
enum { DVP_WEIGHT_NONE = 0, DVP_WEIGHT_RATIO = 1, DVP_WEIGHT_TRUNCATE = 2, DVP_WEIGHT_MASK = 3 };

/*
 * Per-token outputs of one policy ("side"): each pointer is a device array of
 * T elements and may be NULL when the caller does not want it.
 */
typedef struct {
  float *max;       /* m = max_k z_k                                          */
  float *lse;       /* ln sum_k e^{z_k}                  (full vocabulary)    */
  float *lse_safe;  /* ln sum_{k in V_S} e^{z_k}                              */
  float *logp;      /* ln pi(a)                                               */
  float *logp_mp;   /* ln pi^mp(a); -inf when a is pruned      (Def. 5.2)     */
  float *comp_mp;   /* 1 - pi^mp(a), summed without the a term (no cancellation) */
  int32_t *count;   /* |V_S|                                                  */
  uint32_t *mask;   /* [T, ceil(V/32)] packed: bit (k%32) of word k/32 set    */
                    /* when k in V_S; padding bits of the last word are zero  */
  float *log_cov;   /* ln Z, Z = sum_{k in V_S} pi(k) the coverage of Def. 5.2 */
                    /* (<= 0; 1 - Z is the total variation distance between    */
                    /* pi^mp and pi in the proof of Prop. 5.5).  Formed in     */
                    /* double from the two sums the kernel holds, not from the */
                    /* float outputs lse_safe and lse; Z itself is good to      */
                    /* about 1e-5 (float32 sums), so 1 - Z keeps 1e-3 relative  */
                    /* accuracy down to about 1 - Z = 1e-2                      */
} dvp_side_out;

/*
 * dvp_forward -- Def. 5.1, Def. 5.2, Prop. 5.6(1) for the training and the
 * inference logits, the per-token log-ratio of Thm. 5.3 / App. A protocol 4,
 * and, when `upstream` and `grad_train` are both given, the gradient of
 * Prop. 5.4 / Prop. 5.6(2) written in the same sweep over the training row.
 *
 *   train_logits  device [T, ld_train], required
 *   infer_logits  device [T, ld_infer] or NULL (then `infer`, `log_ratio`
 *                 must be NULL); same dtype as the training logits
 *   ids           device [T] int64 or int32; id < 0: statistics only
 *   upstream      device [T] float32: g_t = dLoss / d ln pi^mp_train(a_t)
 *   grad_train    device [T, ld_grad] of grad_dtype: g_t (1[k=a] - pi^mp(k))
 *                 on V_S, 0 off it, the whole row 0 when a is not in V_S;
 *                 rounded to nearest-even in grad_dtype
 *   log_ratio     device [T] float32: ln pi^mp_train(a) - ln pi^mp_infer(a);
 *                 -inf when a is outside V_S (importance ratio zero, remark
 *                 after Thm. 5.3), +inf when a is in V_S but outside V'_S
 *   flags         device [T] bytes, DVP_FLAG_* bits
 *   weight_kind   DVP_WEIGHT_*; other than NONE needs infer_logits, upstream and
 *                 grad_train; weight_lo <= weight_hi, both >= 0, not NaN
 *   weight_out    device [T] float32 or NULL: the weight each token used (NaN
 *                 for a row without a valid sampled id)
 *   launch_hint   0 = library default; otherwise threads per block (a multiple
 *                 of 32, at most 512) in the low 16 bits, a kernel choice in the
 *                 next 8 bits, and the number of blocks that share one row (0, 1, 2
 *                 or 4; a thread-block cluster) in the top 8 bits.  Kernel choice:
 *                 0 or 2 the default kernel (one sweep, then revisits of the 32-byte
 *                 pieces of the row that can hold safe tokens); 3 or 4 (2-byte
 *                 logits, at most 256 threads, no cluster) the kernel that keeps
 *                 the candidates of the safe set in shared memory while the row
 *                 streams and reads nothing twice, with 3 or 4 blocks per SM;
 *                 0x11 (with zero elsewhere) the kernel that keeps the row itself
 *                 in shared memory (rows of up to 480 KB whose byte length is a
 *                 multiple of 16).  Rows a chosen kernel cannot take run the
 *                 default one.  Tuning only: the safe set and counts do not
 *                 depend on it.
 *                 TEST ONLY: 0x1e in the second byte is a self-test of the 0x11
 *                 kernel's wait limit, not an operating mode: its first block
 *                 withholds its first copy, the wait for it runs out after about
 *                 a second, the launch ends by itself with undefined outputs and
 *                 dvp_row_wait_status reports code 1 or 2
 *
 * Rows whose start is 32-byte aligned in all three matrices take the
 * vectorised kernels; any other layout takes a scalar kernel, same results.
 * Needs no workspace.  Errors: DVP_ERR_INVALID_ARG for NULL required
 * pointers, T < 0, V < 1, ld < V, rho outside [0,1] or NaN, upstream without
 * grad_train or the reverse, a malformed launch_hint; DVP_ERR_UNSUPPORTED
 * for unknown dtypes or V >= 2^31 - 256.  Rows too long for the on-chip row
 * summary of the vectorised kernel fall back to the scalar kernel.
 * T = 0 is a valid no-op.
 */
typedef struct {
  uint32_t struct_size;
  int32_t logits_dtype; /* dvp_dtype of train_logits and infer_logits */
  int32_t grad_dtype;   /* dvp_dtype of grad_train                    */
  int32_t id_dtype;     /* dvp_id_dtype                               */
  int64_t T, V;
  int64_t ld_train, ld_infer, ld_grad;
  double rho;
  const void *train_logits;
  const void *infer_logits;
  const void *ids;
  const float *upstream;
  void *grad_train;
  dvp_side_out train;
  dvp_side_out infer;
  float *log_ratio;
  uint8_t *flags;
  void *stream;
  uint32_t launch_hint;
  uint32_t mode;      /* DVP_MODE_* bits */
  float mask_value;   /* used with DVP_MODE_FINITE_MASK */
  uint32_t weight_kind; /* DVP_WEIGHT_* */
  float weight_lo, weight_hi;
  float *weight_out;
} dvp_forward_args;

int dvp_forward(const dvp_forward_args *args);

/*
 * dvp_backward -- Prop. 5.4 / Prop. 5.6(2) as a stand-alone streaming map for
 * callers whose upstream gradient depends on the forward outputs.  Takes the
 * vectors a previous dvp_forward saved for the same logits, ids and rho:
 *
 *   max_t, lse_safe_t, flags   device [T], required (from dvp_forward)
 *   comp_mp_t                  device [T] or NULL; when NULL the a-th entry is
 *                              g (1 - exp(z_a - lse_safe)), which loses digits
 *                              as pi^mp(a) -> 1
 * Reads the training logits once and writes grad_train once.  Same error
 * rules as dvp_forward.  Needs no workspace.
 */
typedef struct {
  uint32_t struct_size;
  int32_t logits_dtype, grad_dtype, id_dtype;
  int64_t T, V;
  int64_t ld_train, ld_grad;
  double rho;
  const void *train_logits;
  const void *ids;
  const float *upstream;
  const float *max_t;
  const float *lse_safe_t;
  const float *comp_mp_t;
  const uint8_t *flags;
  void *grad_train;
  void *stream;
  uint32_t launch_hint;
  uint32_t mode;      /* as in the dvp_forward call that saved the vectors */
  float mask_value;
  uint32_t reserved_;
} dvp_backward_args;

int dvp_backward(const dvp_backward_args *args);

/*
 * dvp_fused_lmhead_forward_backward -- the same objective with the training
 * logits produced on the fly as z = hidden x W_vocab^T (bf16 operands, fp32
 * accumulation on the tensor cores), so the [T, V] training logits are never
 * stored: rows are processed in panels of `panel_rows` tokens whose logits
 * live in the workspace only.  The gradient flows through the linear head by
 * the chain rule of Prop. 5.6(2): d_hidden = G W and d_w = G^T hidden with
 * G = dLoss/dz as in dvp_forward.
 *
 *   hidden        device [T, ld_hidden] bf16
 *   w_vocab       device [V, ld_w] bf16
 *   infer_logits  device [T, ld_infer] bf16 (what the inference engine
 *                 computed for the same parameters), or NULL (then `infer`
 *                 outputs and log_ratio must be NULL)
 *   d_hidden      device [T, ld_dh] float32, overwritten
 *   d_w           device [V, ld_dw] float32; overwritten, or added to when
 *                 accumulate_dw != 0
 *   workspace     device, 256-byte aligned, at least
 *                 dvp_workspace_bytes(DVP_ENTRY_FUSED_LMHEAD, args) bytes.
 *                 Its first 32-bit word is a status: 0 after a run in which
 *                 every tensor-core kernel finished, non-zero if one gave up
 *                 waiting (results are then invalid).
 *   panel_rows    0 = library default (at most 4096); otherwise a multiple of 128
 *   weight_kind   DVP_WEIGHT_NONE, DVP_WEIGHT_TRUNCATE or DVP_WEIGHT_MASK, as in
 *                 dvp_forward: each token's upstream gradient is multiplied by its
 *                 importance weight (needs infer_logits; weight_hi must be finite,
 *                 because the float16 gradient panel is scaled for
 *                 max |upstream| * max(1, weight_hi)); weight_out as in dvp_forward
 *
 * ld_hidden, ld_w, ld_dh, ld_dw must be multiples of 8 and hidden, w_vocab
 * 16-byte, d_hidden, d_w 32-byte aligned (DVP_ERR_UNSUPPORTED otherwise).
 * Membership is decided on the fp32-accumulated logits, so a token whose logit
 * sits within rounding distance of the threshold may fall on either side of
 * the exact-arithmetic decision.  The gradient panel is held in float16 as
 * 2^14 e^{z - max z} on the safe set, the factor of each row (-g / (2^14 s_S))
 * being applied in float32 afterwards: tokens whose probability is below about
 * 4e-9 of the row's largest lose relative accuracy, and hidden states beyond
 * 2047 in magnitude can overflow the float16 copy used for d_w.
 */
typedef struct {
  uint32_t struct_size;
  int32_t id_dtype;
  int64_t T, H, V;
  int64_t ld_hidden, ld_w, ld_infer, ld_dh, ld_dw;
  double rho;
  const void *hidden;
  const void *w_vocab;
  const void *infer_logits;
  const void *ids;
  const float *upstream;
  float *d_hidden;
  float *d_w;
  int32_t accumulate_dw;
  int32_t panel_rows;
  dvp_side_out train;
  dvp_side_out infer;
  float *log_ratio;
  uint8_t *flags;
  void *workspace;
  size_t workspace_bytes;
  void *stream;
  uint32_t weight_kind;
  float weight_lo, weight_hi;
  float *weight_out;
} dvp_fused_args;

int dvp_fused_lmhead_forward_backward(const dvp_fused_args *args);

/*
 * dvp_sequence_aggregate -- sequence-level view of the per-token results: the
 * mismatch of a trajectory is the sum of its token mismatches (Sec. 4.4,
 * Delta_y = sum_t Delta_{a_t}), its importance ratio the product of the token
 * ratios (Thm. 5.3), and a token whose importance weight
 * pi^mp_train / pi^mp_infer = exp(log_ratio) is below `veto_threshold` marks
 * the whole sequence as discarded (App. A, protocol 5; the paper uses 1e-4).
 *
 *   seq_offsets    device [S + 1] int64, non-decreasing; sequence s owns tokens
 *                  [seq_offsets[s], seq_offsets[s+1]), all within [0, T)
 *   log_ratio      device [T] float32 as written by dvp_forward: NaN = token
 *                  without a sampled id (skipped), -inf = outside the training
 *                  safe set (weight zero), +inf = outside the inference set only
 *   seq_log_ratio  device [S]: sum of the token log-ratios; -inf if any token
 *                  has weight zero, else +inf if any token is +inf
 *   min_log_ratio  device [S]: smallest token log-ratio (+inf for an empty sequence)
 *   n_valid        device [S] int32: tokens with a sampled id
 *   n_zero_weight  device [S] int32: tokens with weight zero
 *   veto           device [S] bytes: 1 when some token weight < veto_threshold
 *   log_cov        device [T] float32 or NULL: ln Z per token as written by
 *                  dvp_forward (dvp_side_out.log_cov of the training side)
 *   min_cov        device [S]: min over the sequence's tokens of the coverage Z
 *                  (the Z_min of the bias bound of Prop. 5.5,
 *                  |J_mp - J| <= R_max T (1 - Z_min)); +inf for an empty sequence
 *   mean_cov       device [S]: mean of Z over the sequence's tokens (NaN if empty)
 *                  min_cov and mean_cov need log_cov; every token counts, with
 *                  or without a sampled id.  One sequence spanning [0, T) gives
 *                  the batch-level figures.
 * Each output may be NULL.  veto_threshold >= 0 (0 never vetoes).  S = 0 is a
 * no-op.  Errors: DVP_ERR_INVALID_ARG (null inputs, negative sizes, negative or
 * NaN threshold, min_cov or mean_cov without log_cov).  Offsets are not checked
 * on the device.
 */
typedef struct {
  uint32_t struct_size;
  uint32_t reserved_;
  int64_t T, S;
  const int64_t *seq_offsets;
  const float *log_ratio;
  double veto_threshold;
  float *seq_log_ratio;
  float *min_log_ratio;
  int32_t *n_valid;
  int32_t *n_zero_weight;
  uint8_t *veto;
  void *stream;
  const float *log_cov;
  float *min_cov;
  float *mean_cov;
} dvp_sequence_args;

int dvp_sequence_aggregate(const dvp_sequence_args *args);

/*
 * dvp_monitor -- per-token monitoring quantities over the full vocabulary: the
 * Kullback-Leibler divergences between the inference and the training policy
 * (the training-stability metric of Sec. 6) and the entropy of each (the
 * quantity Sec. 7 proposes to adapt rho to), in nats:
 *   KL(p || q) = sum_k p_k (ln p_k - ln q_k),  H(p) = -sum_k p_k ln p_k,
 *   pi_train = softmax(train_logits[t]), pi_infer = softmax(infer_logits[t]).
 * Both matrices are read once.  Each output is a device [T] float32 array and
 * may be NULL.  Rows that start on 32-byte boundaries take the vectorised
 * kernel, other layouts a scalar one.  Errors as in dvp_forward.
 */
typedef struct {
  uint32_t struct_size;
  int32_t logits_dtype;
  int64_t T, V, ld_train, ld_infer;
  const void *train_logits;
  const void *infer_logits;
  float *kl_infer_train; /* KL(pi_infer || pi_train) */
  float *kl_train_infer; /* KL(pi_train || pi_infer) */
  float *entropy_train;
  float *entropy_infer;
  void *stream;
} dvp_monitor_args;

int dvp_monitor(const dvp_monitor_args *args);

/*
 * dvp_fused_lmhead_forward_backward_static -- the fused entry point for callers
 * that cannot obtain device memory of their own.  (The paper has no counterpart;
 * this is a packaging variant of the entry point above.)
 *
 * Who needs it: code that runs inside a host application which hands out all
 * device memory up front and forbids further allocation, code on a latency
 * critical path where an allocator call (which may synchronise the whole
 * device) is not acceptable, and code that is simply not allowed to own
 * buffers between calls.  Such a caller has the inputs and outputs it was given
 * but no place to put a workspace, and the fused computation cannot run
 * without one.
 *
 * What it does: exactly dvp_fused_lmhead_forward_backward, except that
 * `workspace` and `workspace_bytes` are ignored and the workspace is a fixed
 * array of DVP_STATIC_WORKSPACE_BYTES (32 MiB) that is part of the library
 * image.  Every GPU on which the library's code is loaded holds those 32 MiB
 * until the process exits, whether or not this function is ever called.
 * `panel_rows` = 0 selects 128 here.  The call itself allocates and frees
 * nothing, on the device or through any library.
 *
 * Limit: the workspace the arguments need (dvp_workspace_bytes with the
 * panel_rows this entry uses: pass panel_rows = 128 to that query when you pass 0
 * here, since 0 means up to 4096 there; roughly (2 H + 6 panel_rows) V +
 * 2 H panel_rows bytes) must fit in
 * DVP_STATIC_WORKSPACE_BYTES, e.g. H = 1024, V = 8192, any T up to a few
 * thousand.  Larger problems return DVP_ERR_WORKSPACE and launch nothing.
 * Other errors are those of dvp_fused_lmhead_forward_backward;
 * DVP_ERR_UNSUPPORTED also for a device ordinal of 64 or more.
 *
 * First call on each device: it looks up the array's device address (once per
 * device, with that device current).  Make that first call outside any stream
 * capture.
 *
 * Sharing: all calls on one GPU use the same array, and the array keeps
 * whatever the previous call left in it (the library resets the one word that
 * has to start at zero).  Two calls whose kernels can overlap on the GPU (for
 * instance on different streams) race on it and corrupt each other; issue such
 * calls on one stream, or order them yourself.  After the stream has finished,
 * nothing in the array is needed any more.
 *
 * Status: the ordinary entry point reports a tensor-core kernel that gave up
 * waiting through the first word of the caller's workspace.  Here the caller
 * never sees the workspace, so that word is read with
 * dvp_static_workspace_status: it waits for all work on the current device (it
 * synchronises), then copies the word of the last call on this device to
 * *status_out (a host pointer): 0 = every kernel finished, non-zero = results of
 * that call are invalid.  It allocates nothing either.  Errors:
 * DVP_ERR_INVALID_ARG (NULL), DVP_ERR_CUDA.  Without this call a wait that ran
 * out would go unnoticed (the entry point itself still returns DVP_OK, as
 * launches are asynchronous).
 */
#define DVP_STATIC_WORKSPACE_BYTES (32u * 1024u * 1024u)
int dvp_fused_lmhead_forward_backward_static(const dvp_fused_args *args);
int dvp_static_workspace_status(uint32_t *status_out);

/*
 * dvp_gemm_tn -- the tensor-core contraction the fused entry point is built on,
 * exposed for reuse and testing: C[m, n] (+)= alpha * A[m, k] * B[n, k]^T with A
 * and B both bf16 or both f16 (dtype), row-major with k contiguous, C float32
 * row-major, fp32 accumulation.  The paper has no counterpart; it is the
 * "hidden x W_vocab" product of the LM head and its two transposes.
 *   a, b, c   device; lda, ldb, ldc multiples of 8; a, b 16-byte, c 32-byte aligned
 *   accumulate  bit 0: add to C instead of overwriting it; bit 1: use the kernel that
 *             gives each 128 x 256 tile to one block instead of 256 x 256 tiles to
 *             pairs of blocks (same results up to summation order; for comparison);
 *             bit 2: `a` points to A transposed, [k, m] with m contiguous and row
 *             stride lda (not with bit 1): the tensor cores read it as it lies;
 *             bit 3: every output tile is computed as two halves of the k range
 *             that are added into C with atomics (for few tiles and a long k;
 *             with two addends the sum does not depend on their order)
 *   status    device int32, written non-zero if a kernel gave up waiting
 * Errors: DVP_ERR_INVALID_ARG (null pointers, negative sizes),
 * DVP_ERR_UNSUPPORTED (dtype, alignment), DVP_ERR_CUDA.
 */
int dvp_gemm_tn(const void *a, int64_t lda, const void *b, int64_t ldb, float *c, int64_t ldc,
                int64_t m, int64_t n, int64_t k, int32_t dtype, float alpha, int32_t accumulate,
                int32_t *status, void *stream);

/*
 * dvp_row_wait_status -- the row kernel that keeps rows resident in shared
 * memory (launch_hint stage byte 0x11) waits on hardware barriers for its bulk
 * copies and its block reductions.  Every such wait is bounded; one that runs
 * out ends the launch early (its outputs are then undefined) and ORs a code into a
 * per-device status word: 1 a copy did not land, 2 a ring slot was not handed
 * back, 4 a warp did not reach a block reduction.  This call waits for all work
 * on the current device (it synchronises), copies the word to *status_out (a
 * host pointer) and clears it.  The paper has no counterpart.  0 means that no
 * wait has run out since the last call.  Errors: DVP_ERR_INVALID_ARG (NULL),
 * DVP_ERR_CUDA.
 */
int dvp_row_wait_status(uint32_t *status_out);

/*
 * dvp_debug_bounds_status -- the library can be built a second time with every
 * shared-memory index of the row kernels' on-chip tables and every global element
 * offset they form compared with its extent (python -m paper_2512_23087_b200.build
 * --debug-bounds gives libdvp_b200_bounds.so).  In that build an index out of range
 * is never used: the access is skipped and a code is OR-ed into a per-device word
 * (1 granule-bound table, 2 hot list, 4 granule index, 8 global offset, 16 candidate
 * ring, 32 candidate list, 64 resident slot).  This call waits for all work on the
 * current device, copies the word to *status_out (a host pointer) and clears it; 0
 * means that no check has failed since the last call.  The ordinary build has no
 * checks and returns DVP_ERR_UNSUPPORTED.  The paper has no counterpart: it stands
 * in for a memory checker.  Errors: DVP_ERR_INVALID_ARG (NULL), DVP_ERR_CUDA.
 */
int dvp_debug_bounds_status(uint32_t *status_out);

/*
 * Bytes of device workspace the entry point needs for `args` (a pointer to
 * that entry point's args struct; only sizes and dtypes are read).  Returns 0
 * for entry points that need none and for invalid arguments.
 */
size_t dvp_workspace_bytes(int entry_point, const void *args);

/* Static, human-readable name of a dvp_status value. */
const char *dvp_status_string(int status);

/* Library version, major * 10000 + minor * 100 + patch. */
int dvp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DVP_H_ */
