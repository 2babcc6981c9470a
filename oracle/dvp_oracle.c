/*
 * dvp_oracle.c -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * Plain, slow, fp64 CPU statement of what Dynamic Vocabulary Pruning computes
 * per token row.  It exists so that the CUDA library can be checked against
 * the paper's definitions; only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it.  It shares no code, header, table or constant
 * with the CUDA path.
 *
 * Notation (one row = one state s): logits z in R^V, sampled token a,
 * pruning threshold rho, L = ln(rho), upstream gradient g.
 *
 *   safe set      V_S = { k : pi(k) >= rho * max_j pi(j) }              (Def. 5.1)
 *                     = { k : z_k >= max_j z_j + L }    (App. A, protocol 2; the
 *                       listing prunes with a strict '<', so equality is kept)
 *   coverage      Z   = sum_{k in V_S} pi(k)                            (Def. 5.2)
 *   pruned policy pi^mp(a) = pi(a) / Z  if a in V_S, else 0             (Def. 5.2)
 *   masked logits z_mp,k = z_k on V_S, -inf elsewhere (Sec. 5.5, exact -inf
 *                 semantics; softmax(z_mp) = pi^mp by Prop. 5.6 part 1)
 *   gradient      d log pi^mp(a) / d z_k = 1[k=a] - pi^mp(k) on V_S, 0 off it,
 *                 with the set held fixed (Prop. 5.4, Prop. 5.6 part 2,
 *                 App. A protocol 1); a outside V_S has weight zero
 *                 (remark after Thm. 5.3), so its row of gradients is zero.
 *   log-ratio     r = log pi^mp_train(a) - log pi^mp_infer(a)
 *                 (sign of Delta in Thm. 4.1; App. A protocol 4)
 *
 * Every sum is a Neumaier-compensated fp64 sum taken in index order.
 * Nothing here is blocked, fused or reordered.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_F16 2

/* ---- exact widening of stored logits to double ------------------------- */

static double widen_f32(const void *p, int64_t i) {
  return (double)((const float *)p)[i];
}

static double widen_bf16(const void *p, int64_t i) {
  /* bfloat16 is the upper half of an IEEE binary32 */
  uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
  float f;
  memcpy(&f, &bits, sizeof f);
  return (double)f;
}

static double widen_f16(const void *p, int64_t i) {
  /* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits */
  uint16_t h = ((const uint16_t *)p)[i];
  int sign = (h >> 15) & 1;
  int e = (h >> 10) & 0x1f;
  int f = h & 0x3ff;
  double v;
  if (e == 0)
    v = ldexp((double)f, -24);
  else if (e == 31)
    v = f ? NAN : INFINITY;
  else
    v = ldexp((double)(f + 1024), e - 25);
  return sign ? -v : v;
}

static double widen(const void *p, int dtype, int64_t i) {
  if (dtype == ORACLE_BF16) return widen_bf16(p, i);
  if (dtype == ORACLE_F16) return widen_f16(p, i);
  return widen_f32(p, i);
}

/* ---- compensated accumulation ------------------------------------------ */

typedef struct {
  double sum, comp;
} nsum;

static void nsum_add(nsum *a, double x) {
  double t = a->sum + x;
  if (fabs(a->sum) >= fabs(x))
    a->comp += (a->sum - t) + x;
  else
    a->comp += (x - t) + a->sum;
  a->sum = t;
}

static double nsum_value(const nsum *a) { return a->sum + a->comp; }

/* ---- one side (train or infer) of one row ------------------------------ */

typedef struct {
  double max;        /* m = max_k z_k                                        */
  double lse;        /* ln sum_k e^{z_k}                                     */
  double lse_safe;   /* ln sum_{k in V_S} e^{z_k}                            */
  double log_cov;    /* ln Z = lse_safe - lse                                */
  double logp;       /* ln pi(a)                                             */
  double logp_mp;    /* ln pi^mp(a), -inf when a is pruned                   */
  double sum_safe;   /* sum_{k in V_S} e^{z_k - m}                           */
  double sum_safe_x; /* the same sum without the term k = a                  */
  double tau;        /* m + L                                                */
  int64_t count;     /* |V_S|                                                */
  int32_t member;    /* 1 when a in V_S                                      */
  int32_t pad_;
} oracle_side;

/*
 * z: V doubles.  a < 0 means "no sampled token": the statistics of the row
 * are still produced and the per-token fields are NaN / 0.
 * mask (optional): V bytes, 1 where k is in the safe set.
 */
void dvp_oracle_side(const double *z, int64_t V, int64_t a, double log_rho,
                     oracle_side *out, uint8_t *mask) {
  double m = -INFINITY;
  for (int64_t k = 0; k < V; ++k)
    if (z[k] > m) m = z[k];
  const double tau = m + log_rho;

  nsum all = {0, 0}, safe = {0, 0}, safe_x = {0, 0};
  int64_t n = 0;
  for (int64_t k = 0; k < V; ++k) {
    const double e = exp(z[k] - m);
    const int keep = z[k] >= tau;
    nsum_add(&all, e);
    if (keep) {
      nsum_add(&safe, e);
      if (k != a) nsum_add(&safe_x, e);
      ++n;
    }
    if (mask) mask[k] = (uint8_t)keep;
  }
  const double s = nsum_value(&all), s_safe = nsum_value(&safe);
  out->max = m;
  out->tau = tau;
  out->lse = m + log(s);
  out->lse_safe = m + log(s_safe);
  out->log_cov = log(s_safe) - log(s);
  out->sum_safe = s_safe;
  out->sum_safe_x = nsum_value(&safe_x);
  out->count = n;
  if (a >= 0 && a < V) {
    out->member = z[a] >= tau;
    out->logp = (z[a] - m) - log(s);
    out->logp_mp = out->member ? (z[a] - m) - log(s_safe) : -INFINITY;
  } else {
    out->member = 0;
    out->logp = NAN;
    out->logp_mp = NAN;
  }
}

/*
 * Gradient of g * log pi^mp(a) with respect to the V logits of the row, the
 * safe set held fixed.  The k = a entry is g * (1 - pi^mp(a)) written as
 * g * (sum over V_S without a) / (sum over V_S), which has no cancellation.
 */
void dvp_oracle_side_grad(const double *z, int64_t V, int64_t a, double g,
                          const oracle_side *st, double *grad) {
  if (a < 0 || a >= V || !st->member) {
    for (int64_t k = 0; k < V; ++k) grad[k] = 0.0;
    return;
  }
  for (int64_t k = 0; k < V; ++k) {
    if (z[k] >= st->tau)
      grad[k] = -g * exp(z[k] - st->lse_safe);
    else
      grad[k] = 0.0;
  }
  grad[a] = g * (st->sum_safe_x / st->sum_safe);
}

/*
 * The same statistics with the safe set supplied instead of derived from a
 * threshold: Def. 5.2 and Prop. 5.4 take V_S as given (set: V bytes, 1 where k is
 * in the set).  For logits that exist only up to rounding (the LM-head variant on
 * tensor cores) the set of Def. 5.1 is fixed only up to tokens whose logit sits
 * within rounding distance of the threshold; this form states what every other
 * quantity must be for whichever of those sets was taken.  With the set that
 * dvp_oracle_side itself derives it returns the same numbers.  tau is NaN.
 */
void dvp_oracle_side_given_set(const double *z, int64_t V, int64_t a, const uint8_t *set,
                               oracle_side *out) {
  double m = -INFINITY;
  for (int64_t k = 0; k < V; ++k)
    if (z[k] > m) m = z[k];
  nsum all = {0, 0}, safe = {0, 0}, safe_x = {0, 0};
  int64_t n = 0;
  for (int64_t k = 0; k < V; ++k) {
    const double e = exp(z[k] - m);
    nsum_add(&all, e);
    if (set[k]) {
      nsum_add(&safe, e);
      if (k != a) nsum_add(&safe_x, e);
      ++n;
    }
  }
  const double s = nsum_value(&all), s_safe = nsum_value(&safe);
  out->max = m;
  out->tau = NAN;
  out->lse = m + log(s);
  out->lse_safe = m + log(s_safe);
  out->log_cov = log(s_safe) - log(s);
  out->sum_safe = s_safe;
  out->sum_safe_x = nsum_value(&safe_x);
  out->count = n;
  if (a >= 0 && a < V) {
    out->member = set[a] != 0;
    out->logp = (z[a] - m) - log(s);
    out->logp_mp = out->member ? (z[a] - m) - log(s_safe) : -INFINITY;
  } else {
    out->member = 0;
    out->logp = NAN;
    out->logp_mp = NAN;
  }
}

void dvp_oracle_side_grad_given_set(const double *z, int64_t V, int64_t a, double g,
                                    const uint8_t *set, const oracle_side *st, double *grad) {
  if (a < 0 || a >= V || !st->member) {
    for (int64_t k = 0; k < V; ++k) grad[k] = 0.0;
    return;
  }
  for (int64_t k = 0; k < V; ++k) grad[k] = set[k] ? -g * exp(z[k] - st->lse_safe) : 0.0;
  grad[a] = g * (st->sum_safe_x / st->sum_safe);
}

/*
 * Per-token log-ratio r = ln pi^mp_train(a) - ln pi^mp_infer(a).
 * a outside the training set: the importance ratio is zero (remark after
 * Thm. 5.3), r = -inf whatever the inference side says.  a inside the
 * training set but outside the inference set: r = +inf.
 */
double dvp_oracle_log_ratio(const oracle_side *tr, const oracle_side *inf) {
  if (isnan(tr->logp)) return NAN; /* no sampled token in this row */
  if (!tr->member) return -INFINITY;
  if (!inf->member) return INFINITY;
  return tr->logp_mp - inf->logp_mp;
}

/*
 * Token-level importance weight from the per-token log-ratio r (the factor
 * pi^mp_train(a) / pi^mp_infer(a) of the estimator of Thm. 5.3, formed as the
 * exponential of the difference of log-probabilities, App. A protocol 4), as
 * the comparison methods of Sec. 6 use it per token:
 *   kind 0  no weighting, w = 1
 *   kind 1  the plain ratio, w = e^r
 *   kind 2  truncated importance sampling, w = min(e^r, hi)
 *   kind 3  masked importance sampling, w = e^r if lo <= e^r <= hi, else 0
 * r = -inf (a outside the training safe set) gives w = 0 in every kind; r = +inf
 * (a outside the inference safe set only) gives +inf, hi and 0.  The weight is a
 * constant of the gradient (it is "detached"): the per-token upstream gradient
 * becomes g * w.
 */
double dvp_oracle_token_weight(double r, int kind, double lo, double hi) {
  if (kind == 0) return 1.0;
  if (isnan(r)) return NAN;
  const double w = exp(r);
  if (kind == 1) return w;
  if (kind == 2) return w < hi ? w : hi;
  return (w >= lo && w <= hi) ? w : 0.0;
}

/* ---- batch driver: rows are independent, split statically over threads -- */

typedef struct {
  /* inputs */
  const void *train, *infer; /* [T, ld] stored logits; infer may be NULL   */
  int32_t dtype;             /* ORACLE_F32 / ORACLE_BF16 / ORACLE_F16      */
  int32_t want_mask;         /* fill mask_t / mask_i                        */
  int64_t T, V, ld_train, ld_infer;
  const int64_t *ids;        /* [T]                                         */
  const double *upstream;    /* [T] or NULL                                 */
  double rho;
  /* outputs, each [T] unless noted, each may be NULL */
  oracle_side *side_t, *side_i;
  double *log_ratio;
  double *grad;              /* [T, V] doubles or NULL                      */
  uint8_t *mask_t, *mask_i;  /* [T, V] bytes                                */
  /* token-level importance weighting of the upstream gradient (needs infer) */
  int32_t weight_kind, pad_;
  double weight_lo, weight_hi;
  double *weight;            /* [T] or NULL: the weight each row used       */
} oracle_batch;

typedef struct {
  const oracle_batch *b;
  int64_t row0, row1;
} oracle_job;

static void *oracle_rows(void *arg) {
  const oracle_job *job = (const oracle_job *)arg;
  const oracle_batch *b = job->b;
  const double log_rho = b->rho > 0.0 ? log(b->rho) : -INFINITY;
  double *z = (double *)malloc(sizeof(double) * (size_t)b->V);
  for (int64_t t = job->row0; t < job->row1; ++t) {
    const int64_t a = b->ids ? b->ids[t] : -1;
    oracle_side st, si;
    for (int64_t k = 0; k < b->V; ++k)
      z[k] = widen(b->train, b->dtype, t * b->ld_train + k);
    dvp_oracle_side(z, b->V, a, log_rho, &st,
                    b->want_mask && b->mask_t ? b->mask_t + t * b->V : NULL);
    if (b->side_t) b->side_t[t] = st;
    double w = 1.0;
    if (b->infer) {
      for (int64_t k = 0; k < b->V; ++k)
        z[k] = widen(b->infer, b->dtype, t * b->ld_infer + k);
      dvp_oracle_side(z, b->V, a, log_rho, &si,
                      b->want_mask && b->mask_i ? b->mask_i + t * b->V : NULL);
      if (b->side_i) b->side_i[t] = si;
      const double r = dvp_oracle_log_ratio(&st, &si);
      if (b->log_ratio) b->log_ratio[t] = r;
      w = dvp_oracle_token_weight(r, b->weight_kind, b->weight_lo, b->weight_hi);
      if (b->weight) b->weight[t] = w;
    }
    if (b->grad) {
      for (int64_t k = 0; k < b->V; ++k)
        z[k] = widen(b->train, b->dtype, t * b->ld_train + k);
      const double g = b->upstream ? b->upstream[t] : 0.0;
      /* a row without a sampled token has no weight (NaN) and no gradient */
      dvp_oracle_side_grad(z, b->V, a, (b->weight_kind && !isnan(w)) ? g * w : g, &st,
                           b->grad + t * b->V);
    }
  }
  free(z);
  return NULL;
}

/* Returns the number of threads used. */
int dvp_oracle_batch(const oracle_batch *b, int nthreads) {
  if (nthreads < 1) nthreads = 1;
  if (nthreads > b->T) nthreads = b->T > 0 ? (int)b->T : 1;
  if (nthreads > 1024) nthreads = 1024;
  oracle_job jobs[1024];
  pthread_t tid[1024];
  const int64_t per = (b->T + nthreads - 1) / nthreads;
  for (int i = 0; i < nthreads; ++i) {
    jobs[i].b = b;
    jobs[i].row0 = per * i < b->T ? per * i : b->T;
    jobs[i].row1 = per * (i + 1) < b->T ? per * (i + 1) : b->T;
  }
  if (nthreads == 1) {
    oracle_rows(&jobs[0]);
    return 1;
  }
  for (int i = 0; i < nthreads; ++i)
    pthread_create(&tid[i], NULL, oracle_rows, &jobs[i]);
  for (int i = 0; i < nthreads; ++i) pthread_join(tid[i], NULL);
  return nthreads;
}

/*
 * The masking of the App. A listing, taken literally: pruned logits are not
 * removed but replaced by a finite mask value (Sec. 5.5: "-50.0 in BF16"), which
 * stays in the partition sum, and the threshold max + log(rho) is rounded to the
 * logits' storage type before the strict comparison `logit < threshold`.
 *   u_k = z_k if z_k >= thr else mask_value;  result = log_softmax(u)[a]
 * The gradient flows only through kept positions (the mask value is a constant
 * of `where`), the pruned ones get zero.  `thr` and `mask_value` arrive already
 * rounded to the storage type by the caller.
 */
typedef struct {
  double max, lse_full, lse_masked, logp_masked, comp; /* comp = 1 - softmax(u)_a */
  int64_t count;                                        /* kept tokens            */
  int32_t member, pad_;
} oracle_listing;

void dvp_oracle_listing(const double *z, int64_t V, int64_t a, double thr, double mask_value,
                        double g, oracle_listing *out, double *grad) {
  double m = -INFINITY;
  for (int64_t k = 0; k < V; ++k)
    if (z[k] > m) m = z[k];
  const double top = m > mask_value ? m : mask_value;
  nsum all = {0, 0}, masked = {0, 0}, masked_x = {0, 0};
  int64_t n = 0;
  for (int64_t k = 0; k < V; ++k) {
    const int keep = !(z[k] < thr);
    const double u = keep ? z[k] : mask_value;
    nsum_add(&all, exp(z[k] - m));
    nsum_add(&masked, exp(u - top));
    if (k != a) nsum_add(&masked_x, exp(u - top));
    n += keep;
  }
  const double s = nsum_value(&masked);
  out->max = m;
  out->lse_full = m + log(nsum_value(&all));
  out->lse_masked = top + log(s);
  out->count = n;
  if (a >= 0 && a < V) {
    const int keep_a = !(z[a] < thr);
    out->member = keep_a;
    out->logp_masked = (keep_a ? z[a] : mask_value) - out->lse_masked;
    out->comp = nsum_value(&masked_x) / s;
  } else {
    out->member = 0;
    out->logp_masked = NAN;
    out->comp = NAN;
  }
  if (grad) {
    for (int64_t k = 0; k < V; ++k) {
      const int keep = !(z[k] < thr);
      grad[k] = (a >= 0 && a < V && keep) ? -g * exp(z[k] - out->lse_masked) : 0.0;
    }
    if (a >= 0 && a < V && out->member) grad[a] = g * out->comp;
  }
}

/*
 * Monitoring quantities of one token: the Kullback-Leibler divergences between
 * the full-vocabulary inference and training policies (the stability metric of
 * Sec. 6) and their entropies (the quantity Sec. 7 proposes to adapt rho to).
 *   KL(p || q) = sum_k p_k (ln p_k - ln q_k),   H(p) = - sum_k p_k ln p_k,
 * with p = softmax(z), written out term by term.
 * out: kl_infer_train, kl_train_infer, entropy_train, entropy_infer.
 */
void dvp_oracle_monitor(const double *z, const double *zi, int64_t V, double *out) {
  double m = -INFINITY, mi = -INFINITY;
  for (int64_t k = 0; k < V; ++k) {
    if (z[k] > m) m = z[k];
    if (zi[k] > mi) mi = zi[k];
  }
  nsum s = {0, 0}, si = {0, 0};
  for (int64_t k = 0; k < V; ++k) {
    nsum_add(&s, exp(z[k] - m));
    nsum_add(&si, exp(zi[k] - mi));
  }
  const double lse = m + log(nsum_value(&s)), lsei = mi + log(nsum_value(&si));
  nsum kl_it = {0, 0}, kl_ti = {0, 0}, h_t = {0, 0}, h_i = {0, 0};
  for (int64_t k = 0; k < V; ++k) {
    const double lp = z[k] - lse, lq = zi[k] - lsei; /* ln pi_train(k), ln pi_infer(k) */
    const double p = exp(lp), q = exp(lq);
    if (q > 0) nsum_add(&kl_it, q * (lq - lp));
    if (p > 0) nsum_add(&kl_ti, p * (lp - lq));
    if (p > 0) nsum_add(&h_t, -p * lp);
    if (q > 0) nsum_add(&h_i, -q * lq);
  }
  out[0] = nsum_value(&kl_it);
  out[1] = nsum_value(&kl_ti);
  out[2] = nsum_value(&h_t);
  out[3] = nsum_value(&h_i);
}

int dvp_oracle_sizeof_listing(void) { return (int)sizeof(oracle_listing); }

/*
 * Sequence level (Sec. 4.4: Delta_y = sum_t Delta_{a_t}; Thm. 5.3: the ratio of a
 * trajectory is the product of its token ratios; App. A protocol 5: a token whose
 * importance weight pi^mp_train / pi^mp_infer falls below the veto threshold
 * discards the whole sequence).  Tokens of sequence s are [off[s], off[s+1]).
 * A token without a sampled id (NaN log-ratio) is skipped.  A token outside the
 * training safe set has weight zero: the sequence sum is -inf whatever else it
 * holds, and the sequence is vetoed for any positive threshold.
 */
void dvp_oracle_sequences(const double *log_ratio, const int64_t *off, int64_t S,
                          double veto_threshold, double *seq_log_ratio, double *min_log_ratio,
                          int64_t *n_valid, int64_t *n_zero_weight, uint8_t *veto) {
  for (int64_t s = 0; s < S; ++s) {
    nsum acc = {0, 0};
    double lo = INFINITY;
    int64_t valid = 0, zero = 0;
    int has_pinf = 0, vetoed = 0;
    for (int64_t t = off[s]; t < off[s + 1]; ++t) {
      const double r = log_ratio[t];
      if (isnan(r)) continue;
      ++valid;
      if (r < lo) lo = r;
      if (exp(r) < veto_threshold) vetoed = 1;
      if (isinf(r)) {
        if (r < 0) ++zero; else has_pinf = 1;
      } else {
        nsum_add(&acc, r);
      }
    }
    seq_log_ratio[s] = zero ? -INFINITY : (has_pinf ? INFINITY : nsum_value(&acc));
    min_log_ratio[s] = lo;
    n_valid[s] = valid;
    n_zero_weight[s] = zero;
    veto[s] = (uint8_t)vetoed;
  }
}

/*
 * Coverage statistics of a sequence of states: Z_t = e^{ln Z_t} (Def. 5.2), its
 * minimum over the sequence (the Z_min of Prop. 5.5's bound
 * |J_mp - J| <= R_max T (1 - Z_min)) and its mean.  Empty sequence: +inf and NaN.
 */
void dvp_oracle_coverage(const double *log_cov, const int64_t *off, int64_t S, double *min_cov,
                         double *mean_cov) {
  for (int64_t s = 0; s < S; ++s) {
    nsum acc = {0, 0};
    double lo = INFINITY;
    for (int64_t t = off[s]; t < off[s + 1]; ++t) {
      const double z = exp(log_cov[t]);
      if (z < lo) lo = z;
      nsum_add(&acc, z);
    }
    const int64_t n = off[s + 1] - off[s];
    min_cov[s] = lo;
    mean_cov[s] = n > 0 ? nsum_value(&acc) / (double)n : NAN;
  }
}

int dvp_oracle_sizeof_side(void) { return (int)sizeof(oracle_side); }
int dvp_oracle_sizeof_batch(void) { return (int)sizeof(oracle_batch); }
