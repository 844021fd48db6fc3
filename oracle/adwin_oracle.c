/*
 * adwin_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, float64 CPU statement of what the windowed on-policy-distillation (OPD)
 * divergence path computes.  It exists so that the CUDA library can be checked against
 * something that can be compared with the paper by eye.  Only the test-suite, the smoke check
 * and the benchmark's CPU-baseline leg may call it.  It shares no code, header, table or
 * constant with the CUDA path and is never used as a fallback.
 *
 * Notation (paper, Section 2.1 and 2.3): for one response position (b,t)
 *   z = student logits over the vocabulary,  u = teacher logits,  y = sampled token,
 *   p = softmax(z) = pi_theta(. | x, y_<t),  q = softmax(u) = pi_phi(. | x, y_<t).
 *
 * Pins (see tests/test_oracle_*.py): lse/log-softmax against scipy and torch float64; KL against
 * KL(p||p)=0, KL>=0, shift invariance, uniform / one-hot / V=2 closed forms, exact rational
 * enumeration at tiny V, a hand-computed two-point example fixing the direction; c against
 * E_{y~p}[c]=KL; gradients against central finite differences, zero row sum and the
 * expectation identity of Appendix A.1; window mask against brute-force prefix sums;
 * rho/SNR/L_next against closed forms, hand tables and a literal dot-product cosine.
 * The fused LM-head form (logits = hidden states times an output embedding; oracle functions in
 * adwin_oracle.py, which call the per-row definition below on float64 logits) is pinned in
 * tests/test_oracle_lmhead.py: explicit loops for the products, equality with this file's batch
 * function on exactly representable logits, central differences with respect to hidden states and
 * LM-head weight, nothing from positions outside the window, and the LM-head-weight-space cosine
 * against its Gram form, the orthonormal case (= logit-space rho) and the shared-hidden-state case.
 * The cosine of Section 4.2 over ALL model parameters (gradients in R^d through the whole model's
 * Jacobian) is NOT computed here: parity unpinned for that quantity (out of scope: it needs a
 * model); the LM-head weight is the one parameter block this path can see.
 *
 * No blocking, fusion or reordering: every function below is the definition written out.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_F64 2 /* logits that are already double (formed from hidden states and an LM head) */

#define ORACLE_MODE_FULL_KL 0 /* gradient of the per-token reverse KL of Eq. 2 */
#define ORACLE_MODE_SAMPLED 1 /* gamma = 0 score-function estimator, Eq. 4 */

#define ORACLE_FLAG_ZERO_TAIL 1
#define ORACLE_FLAG_RANGE_FULL 2

#define ORACLE_ALIGN_DEGENERATE 1
#define ORACLE_ALIGN_NONE_ADMISSIBLE 2

/* Exact widening of a stored logit to double. */
static double load_logit(const void *base, int dtype, int64_t idx) {
  if (dtype == ORACLE_F32) {
    return (double)((const float *)base)[idx];
  } else if (dtype == ORACLE_F64) {
    return ((const double *)base)[idx];
  } else {
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
  }
}

/* Neumaier compensated running sum: sum += x. */
static void comp_add(double *sum, double *comp, double x) {
  double t = *sum + x;
  if (fabs(*sum) >= fabs(x))
    *comp += (*sum - t) + x;
  else
    *comp += (x - t) + *sum;
  *sum = t;
}

/* log sum_k exp(v_k), two passes (max, then sum), no online trick. */
double adwin_oracle_logsumexp(const double *v, int64_t V) {
  double m = -INFINITY;
  for (int64_t k = 0; k < V; ++k)
    if (v[k] > m) m = v[k];
  if (!(m > -INFINITY)) return m; /* empty or all -inf */
  double s = 0.0, c = 0.0;
  for (int64_t k = 0; k < V; ++k) comp_add(&s, &c, exp(v[k] - m));
  return m + log(s + c);
}

/*
 * One response position.
 *   kl      = sum_k p_k (log p_k - log q_k)                 per-token form of Eq. 2 (student first)
 *   c       = log p_y - log q_y                             step-wise cost c_t, Section 2.3
 *   g (FULL_KL) = alpha * p_k ((log p_k - log q_k) - kl)    d kl / d z_k
 *   g (SAMPLED) = alpha * c (1[k=y] - p_k)                  c_t * d log p_y / d z_k, Eq. 4
 *   gsq     = sum_k g_k^2, summed directly from g
 * 0 * log 0 is taken as 0.  y outside [0,V) gives c = NaN (and a NaN SAMPLED gradient).
 * g may be NULL (gsq is still produced).
 */
void adwin_oracle_row(const double *z, const double *u, int64_t V, int64_t y, double alpha,
                      int mode, double *kl, double *c, double *lse_s, double *lse_t,
                      double *gsq, double *g) {
  double ls = adwin_oracle_logsumexp(z, V);
  double lt = adwin_oracle_logsumexp(u, V);
  double acc = 0.0, comp = 0.0;
  for (int64_t k = 0; k < V; ++k) {
    double lp = z[k] - ls;
    double lq = u[k] - lt;
    double p = exp(lp);
    if (p != 0.0) comp_add(&acc, &comp, p * (lp - lq));
  }
  double KL = acc + comp;
  double cost = (y >= 0 && y < V) ? (z[y] - ls) - (u[y] - lt) : NAN;

  double q2 = 0.0, q2c = 0.0;
  for (int64_t k = 0; k < V; ++k) {
    double lp = z[k] - ls;
    double lq = u[k] - lt;
    double p = exp(lp);
    double gk;
    if (mode == ORACLE_MODE_FULL_KL) {
      gk = (p != 0.0) ? alpha * p * ((lp - lq) - KL) : 0.0;
    } else {
      gk = alpha * cost * ((k == y ? 1.0 : 0.0) - p);
    }
    if (g) g[k] = gk;
    comp_add(&q2, &q2c, gk * gk);
  }
  *kl = KL;
  *c = cost;
  *lse_s = ls;
  *lse_t = lt;
  *gsq = q2 + q2c;
}

/*
 * The whole batch.  Logits are [B,T,V] with row stride ld (elements); tokens [B,T];
 * window [B] = W_b; rollout_len [B] = R_b (NULL => T).
 * A position t of sequence b is inside the prefix window when t < W_b and t < R_b and t < T
 * (Section 4.1: the loss is evaluated on the prefix of length L_t; a rollout that ended early
 * has fewer tokens).  With ORACLE_FLAG_RANGE_FULL the per-token scalars are produced for every
 * t < R_b (the delayed full-rollout probe, Section 4.2) while the gradient is still written only
 * inside the window.  Per-token outputs of positions that are not processed are 0.  Gradient rows
 * outside the window are left untouched unless ORACLE_FLAG_ZERO_TAIL, which zero-fills them.
 * grad (double, row stride ld_grad) may be NULL.  lse outputs may be NULL.
 * Returns 0, or 5 when a window / rollout length is negative or R_b > T.
 */
int adwin_oracle_opd_kl_fwd_bwd(const void *student, const void *teacher, int dtype, int64_t B,
                                int64_t T, int64_t V, int64_t ld, const int32_t *tokens,
                                const int32_t *window, const int32_t *rollout_len,
                                double grad_scale, int grad_mode, int flags, double *grad,
                                int64_t ld_grad, double *kl, double *logratio, double *gsq,
                                double *lse_student, double *lse_teacher) {
  for (int64_t b = 0; b < B; ++b) {
    int64_t R = rollout_len ? rollout_len[b] : T;
    if (window[b] < 0 || R < 0 || R > T) return 5;
  }
  int64_t rows = B * T;
#ifdef _OPENMP
#pragma omp parallel
#endif
  {
    double *z = (double *)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
    double *u = (double *)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
    double *g = (double *)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
    for (int64_t r = 0; r < rows; ++r) {
      int64_t b = r / T, t = r % T;
      int64_t W = window[b];
      int64_t R = rollout_len ? rollout_len[b] : T;
      /* brute-force membership, no precomputed effective window */
      int in_window = (t < W) && (t < R) && (t < T);
      int in_rollout = (t < R) && (t < T);
      int processed = (flags & ORACLE_FLAG_RANGE_FULL) ? in_rollout : in_window;
      double o_kl = 0, o_c = 0, o_ls = 0, o_lt = 0, o_gsq = 0;
      if (processed) {
        for (int64_t k = 0; k < V; ++k) {
          z[k] = load_logit(student, dtype, r * ld + k);
          u[k] = load_logit(teacher, dtype, r * ld + k);
        }
        adwin_oracle_row(z, u, V, tokens[r], grad_scale, grad_mode, &o_kl, &o_c, &o_ls, &o_lt,
                         &o_gsq, g);
      }
      kl[r] = o_kl;
      logratio[r] = o_c;
      gsq[r] = o_gsq;
      if (lse_student) lse_student[r] = o_ls;
      if (lse_teacher) lse_teacher[r] = o_lt;
      if (grad) {
        if (processed && in_window) {
          for (int64_t k = 0; k < V; ++k) grad[r * ld_grad + k] = g[k];
        } else if (flags & ORACLE_FLAG_ZERO_TAIL) {
          for (int64_t k = 0; k < V; ++k) grad[r * ld_grad + k] = 0.0;
        }
      }
    }
    free(z);
    free(u);
    free(g);
  }
  return 0;
}

/*
 * Windowed sums (the loss "on this prefix", Section 4.1): per sequence over the positions that
 * are inside the window, seq_out[b] = { sum kl, sum c, sum gsq, number of positions };
 * batch_out = the same four summed over sequences.
 */
void adwin_oracle_window_reduce(const double *kl, const double *logratio, const double *gsq,
                                const int32_t *window, const int32_t *rollout_len, int64_t B,
                                int64_t T, double *seq_out, double *batch_out) {
  double tot[4] = {0, 0, 0, 0};
  for (int64_t b = 0; b < B; ++b) {
    int64_t W = window[b];
    int64_t R = rollout_len ? rollout_len[b] : T;
    double s[4] = {0, 0, 0, 0};
    for (int64_t t = 0; t < T; ++t) {
      if (t < W && t < R) {
        s[0] += kl[b * T + t];
        s[1] += logratio[b * T + t];
        s[2] += gsq ? gsq[b * T + t] : 0.0;
        s[3] += 1.0;
      }
    }
    for (int i = 0; i < 4; ++i) {
      seq_out[b * 4 + i] = s[i];
      tot[i] += s[i];
    }
  }
  for (int i = 0; i < 4; ++i) batch_out[i] = tot[i];
}

/*
 * Prefix-versus-full alignment audit (Section 4.2) in logit space.
 *
 * In logit space every (b,t,k) is its own coordinate and the prefix gradient u^(L) is the
 * full-rollout gradient u^probe with the rows t >= L zeroed, so <u^(L), u^probe> = |u^(L)|^2 and
 *   rho(L) = cos(u^probe, u^(L)) = |u^(L)| / |u^probe| = sqrt(Q(L) / Q_full),
 * with Q(L) = sum of gsq over t < min(L, R_b).  adwin_oracle_literal_cosine() below checks this
 * against the dot product on materialised tensors.
 *
 * Slots j = 0..K-1 are the candidate lengths, slot K is the sequence's own window W_b.
 *   seq_stats[b][j]  = { Q_b(L_j), sum kl, sum c over the same prefix, rho_b(L_j) }
 *   seq_full[b]      = { Q_b_full, sum kl, sum c over t < R_b }
 *   batch_stats[j]   = { rho_micro, rho_macro, snr_micro, admissible (0/1), n_tokens }
 * macro = mean over all B sequences of rho_b (per-sample cosines averaged); micro = the cosine
 * after summing over the batch (Figure 5).  SNR = rho^2 / (1 - rho^2); admissible when
 * rho_micro >= rho_star (threshold equation of Section 4.2, inclusive).  L_next = the smallest candidate length that is
 * admissible (Section 4.2); when none is, the largest candidate and flag NONE_ADMISSIBLE.
 * A zero full norm gives rho = 1 (prefix and full gradients coincide) and flag DEGENERATE.
 */
void adwin_oracle_probe_align(const double *kl, const double *logratio, const double *gsq,
                              const int32_t *window, const int32_t *rollout_len, int64_t B,
                              int64_t T, const int32_t *candidates, int32_t K, double rho_star,
                              double *seq_stats, double *seq_full, double *batch_stats,
                              int32_t *L_next, int32_t *flags_out) {
  int flags = 0;
  for (int64_t b = 0; b < B; ++b) {
    int64_t R = rollout_len ? rollout_len[b] : T;
    double f[3] = {0, 0, 0};
    for (int64_t t = 0; t < T; ++t)
      if (t < R) {
        f[0] += gsq[b * T + t];
        f[1] += kl[b * T + t];
        f[2] += logratio[b * T + t];
      }
    for (int i = 0; i < 3; ++i) seq_full[b * 3 + i] = f[i];
    for (int32_t j = 0; j <= K; ++j) {
      int64_t L = (j < K) ? candidates[j] : window[b];
      double s[3] = {0, 0, 0};
      for (int64_t t = 0; t < T; ++t)
        if (t < L && t < R) {
          s[0] += gsq[b * T + t];
          s[1] += kl[b * T + t];
          s[2] += logratio[b * T + t];
        }
      double rho;
      if (f[0] > 0.0) {
        rho = sqrt(s[0] / f[0]);
      } else {
        rho = 1.0;
        flags |= ORACLE_ALIGN_DEGENERATE;
      }
      double *o = seq_stats + ((b * (K + 1)) + j) * 4;
      o[0] = s[0];
      o[1] = s[1];
      o[2] = s[2];
      o[3] = rho;
    }
  }
  for (int32_t j = 0; j <= K; ++j) {
    double qp = 0, qf = 0, macro = 0, ntok = 0;
    for (int64_t b = 0; b < B; ++b) {
      int64_t R = rollout_len ? rollout_len[b] : T;
      int64_t L = (j < K) ? candidates[j] : window[b];
      qp += seq_stats[((b * (K + 1)) + j) * 4 + 0];
      qf += seq_full[b * 3 + 0];
      macro += seq_stats[((b * (K + 1)) + j) * 4 + 3];
      ntok += (double)(L < R ? L : R);
    }
    double micro;
    if (qf > 0.0) {
      micro = sqrt(qp / qf);
    } else {
      micro = 1.0;
      flags |= ORACLE_ALIGN_DEGENERATE;
    }
    double r2 = micro * micro;
    double *o = batch_stats + j * 5;
    o[0] = micro;
    o[1] = (B > 0) ? macro / (double)B : 1.0;
    o[2] = (r2 < 1.0) ? r2 / (1.0 - r2) : INFINITY;
    o[3] = (micro >= rho_star) ? 1.0 : 0.0;
    o[4] = ntok;
  }
  int32_t best = -1, largest = -1;
  for (int32_t j = 0; j < K; ++j) {
    if (candidates[j] > largest) largest = candidates[j];
    if (batch_stats[j * 5 + 3] != 0.0 && (best < 0 || candidates[j] < best)) best = candidates[j];
  }
  if (best < 0) {
    best = largest;
    flags |= ORACLE_ALIGN_NONE_ADMISSIBLE;
  }
  *L_next = best;
  *flags_out = flags;
}

/*
 * Literal cosine between a prefix gradient and the full-rollout gradient, from materialised
 * tensors (tiny shapes only).  grad is [B,T,V] double holding the gradient of every position
 * t < R_b.  per_seq[b] = cosine for sequence b alone; the return value is the cosine after
 * concatenating all sequences (batch aggregation in logit space).
 */
double adwin_oracle_literal_cosine(const double *grad, const int32_t *rollout_len, int64_t B,
                                   int64_t T, int64_t V, int64_t L, double *per_seq) {
  double dot_all = 0, np_all = 0, nf_all = 0;
  for (int64_t b = 0; b < B; ++b) {
    int64_t R = rollout_len ? rollout_len[b] : T;
    double dot = 0, np = 0, nf = 0;
    for (int64_t t = 0; t < T; ++t)
      for (int64_t k = 0; k < V; ++k) {
        double full = (t < R) ? grad[(b * T + t) * V + k] : 0.0;
        double pre = (t < L && t < R) ? grad[(b * T + t) * V + k] : 0.0;
        dot += pre * full;
        np += pre * pre;
        nf += full * full;
      }
    if (per_seq) per_seq[b] = (nf > 0) ? (np > 0 ? dot / (sqrt(np) * sqrt(nf)) : 0.0) : 1.0;
    dot_all += dot;
    np_all += np;
    nf_all += nf;
  }
  if (!(nf_all > 0)) return 1.0;
  return (np_all > 0) ? dot_all / (sqrt(np_all) * sqrt(nf_all)) : 0.0;
}

/*
 * Discounted return-to-go of the per-token costs (Eq. 3; G_t^gamma in the appendix that derives the
 * OPD gradient), written out as the definition: for every position t inside the range,
 *   G[b,t] = sum over t' from t to the last position of the range of gamma^(t'-t) * c[b,t'],
 * one power and one product per term, no recurrence.  The range is the prefix window (t < W_b,
 * t < R_b, t < T) or, with ORACLE_FLAG_RANGE_FULL, the rollout (t < R_b, t < T); positions outside
 * it get 0.  gamma^0 = 1 also for gamma = 0 (C's pow), which gives G = c, the token-local case.
 */
void adwin_oracle_return_to_go(const double *c, const int32_t *window, const int32_t *rollout_len,
                               int64_t B, int64_t T, double gamma, int flags, double *G) {
  for (int64_t b = 0; b < B; ++b) {
    int64_t W = window[b];
    int64_t R = rollout_len ? rollout_len[b] : T;
    for (int64_t t = 0; t < T; ++t) {
      int in_t = (flags & ORACLE_FLAG_RANGE_FULL) ? (t < R && t < T) : (t < W && t < R && t < T);
      double acc = 0.0, comp = 0.0;
      if (in_t) {
        for (int64_t tp = t; tp < T; ++tp) {
          int in_tp = (flags & ORACLE_FLAG_RANGE_FULL) ? (tp < R) : (tp < W && tp < R);
          if (!in_tp) break;
          comp_add(&acc, &comp, pow(gamma, (double)(tp - t)) * c[b * T + tp]);
        }
      }
      G[b * T + t] = acc + comp;
    }
  }
}

/*
 * One position of the future-coupled estimator in logit space (Eq. 3): the sampled-token gradient
 * of Eq. 4 with a given coefficient w in place of c_t,
 *   g_k = alpha * w * (1[k = y] - p_k),    p = softmax(z),    gsq = sum_k g_k^2.
 * y outside [0,V) gives a NaN gradient, like the SAMPLED mode of adwin_oracle_row.
 */
void adwin_oracle_row_weighted(const double *z, int64_t V, int64_t y, double alpha, double w,
                               double *gsq, double *g) {
  double ls = adwin_oracle_logsumexp(z, V);
  double coef = (y >= 0 && y < V) ? alpha * w : NAN;
  double q2 = 0.0, q2c = 0.0;
  for (int64_t k = 0; k < V; ++k) {
    double p = exp(z[k] - ls);
    double gk = coef * ((k == y ? 1.0 : 0.0) - p);
    if (g) g[k] = gk;
    comp_add(&q2, &q2c, gk * gk);
  }
  *gsq = q2 + q2c;
}

/*
 * Teacher-side drift of one position (Section 3.1): the entropy of the teacher distribution
 * q = softmax(u), H = - sum_k q_k log q_k (0 log 0 = 0), whose exponential is the teacher
 * branching factor BF, and the rank of the sampled token under q: 1 + the number of entries with a
 * strictly larger logit.  y outside [0,V) gives rank 0.
 */
void adwin_oracle_teacher_drift_row(const double *u, int64_t V, int64_t y, double *entropy,
                                    int64_t *rank) {
  double lt = adwin_oracle_logsumexp(u, V);
  double acc = 0.0, comp = 0.0;
  int64_t above = 0;
  for (int64_t k = 0; k < V; ++k) {
    double lq = u[k] - lt;
    double q = exp(lq);
    if (q != 0.0) comp_add(&acc, &comp, -q * lq);
    if (y >= 0 && y < V && u[k] > u[y]) ++above;
  }
  *entropy = acc + comp;
  *rank = (y >= 0 && y < V) ? above + 1 : 0;
}

/*
 * The survival fraction S_T^(k) of Section 3.1, literally: for every position T' (0-based) the
 * fraction of the B rollouts in which every position t <= T' that belongs to the rollout
 * (t < R_b) has rank <= k.  rank is [B,T] (entries past the rollout are ignored).
 */
void adwin_oracle_topk_survival(const int64_t *rank, const int32_t *rollout_len, int64_t B,
                                int64_t T, int64_t k, double *survival) {
  for (int64_t tp = 0; tp < T; ++tp) {
    int64_t alive = 0;
    for (int64_t b = 0; b < B; ++b) {
      int64_t R = rollout_len ? rollout_len[b] : T;
      int ok = 1;
      for (int64_t t = 0; t <= tp && t < R; ++t)
        if (rank[b * T + t] > k) ok = 0;
      alive += ok;
    }
    survival[tp] = (double)alive / (double)B;
  }
}

/*
 * Scale of the terms that a ONE-sweep evaluation of gsq adds and subtracts (a conditioning
 * measure for tests, not a quantity of the method).  Without a second sweep the squared norm
 * sum_k p_k^2 (delta_k - E_p delta)^2, delta = z - u, can only be accumulated about a centre that
 * is known beforehand -- the sampled token's delta_y -- and corrected afterwards:
 *   sum p^2 (delta - delta_y)^2 - 2 c0 sum p^2 (delta - delta_y) + c0^2 sum p^2,  c0 = E_p delta - delta_y.
 * Each of the three sums is bounded by  2 sum_k p_k^2 [ (delta_k - delta_y)^2 + c0^2 ],  which is what
 * this returns (times alpha^2).  On a peaked row with an off-peak sample it exceeds gsq by orders
 * of magnitude, and a float32 evaluation then keeps correspondingly fewer digits of gsq.
 * SAMPLED mode: gsq = (alpha c)^2 [ (1 - p_y)^2 + sum_{k != y} p_k^2 ] is evaluated as
 * sum p^2 - p_y^2 + (1 - p_y)^2; the scale returned is (alpha c)^2 [ sum p^2 + p_y^2 + (1 - p_y)^2 ].
 * y outside [0,V): the centre is delta_0 (FULL_KL), the result NaN (SAMPLED).
 */
double adwin_oracle_gsq_term_scale(const double *z, const double *u, int64_t V, int64_t y,
                                   double alpha, int mode) {
  double ls = adwin_oracle_logsumexp(z, V);
  double lt = adwin_oracle_logsumexp(u, V);
  int ok = (y >= 0 && y < V);
  double dy = ok ? z[y] - u[y] : z[0] - u[0];
  double mean = 0.0, mc = 0.0;
  for (int64_t k = 0; k < V; ++k) comp_add(&mean, &mc, exp(z[k] - ls) * (z[k] - u[k]));
  double c0 = (mean + mc) - dy;
  double acc = 0.0, comp = 0.0, p2 = 0.0, p2c = 0.0;
  for (int64_t k = 0; k < V; ++k) {
    double p = exp(z[k] - ls);
    double d = (z[k] - u[k]) - dy;
    comp_add(&acc, &comp, p * p * (d * d + c0 * c0));
    comp_add(&p2, &p2c, p * p);
  }
  if (mode == ORACLE_MODE_FULL_KL) return 2.0 * alpha * alpha * (acc + comp);
  if (!ok) return NAN;
  double py = exp(z[y] - ls);
  double c = (z[y] - ls) - (u[y] - lt);
  return alpha * alpha * c * c * ((p2 + p2c) + py * py + (1.0 - py) * (1.0 - py));
}

/* The same for every processed position of a batch (0 elsewhere); arguments as in
 * adwin_oracle_opd_kl_fwd_bwd. */
int adwin_oracle_gsq_term_scale_batch(const void *student, const void *teacher, int dtype,
                                      int64_t B, int64_t T, int64_t V, int64_t ld,
                                      const int32_t *tokens, const int32_t *window,
                                      const int32_t *rollout_len, double grad_scale, int grad_mode,
                                      int flags, double *scale) {
  for (int64_t b = 0; b < B; ++b) {
    int64_t R = rollout_len ? rollout_len[b] : T;
    if (window[b] < 0 || R < 0 || R > T) return 5;
  }
  int64_t rows = B * T;
#ifdef _OPENMP
#pragma omp parallel
#endif
  {
    double *z = (double *)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
    double *u = (double *)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
    for (int64_t r = 0; r < rows; ++r) {
      int64_t b = r / T, t = r % T;
      int64_t R = rollout_len ? rollout_len[b] : T;
      int in_window = (t < window[b]) && (t < R) && (t < T);
      int in_rollout = (t < R) && (t < T);
      int processed = (flags & ORACLE_FLAG_RANGE_FULL) ? in_rollout : in_window;
      double v = 0.0;
      if (processed) {
        for (int64_t k = 0; k < V; ++k) {
          z[k] = load_logit(student, dtype, r * ld + k);
          u[k] = load_logit(teacher, dtype, r * ld + k);
        }
        v = adwin_oracle_gsq_term_scale(z, u, V, tokens[r], grad_scale, grad_mode);
      }
      scale[r] = v;
    }
    free(z);
    free(u);
  }
  return 0;
}

int adwin_oracle_num_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
