/*
 * adwin.h -- C ABI of the B200 (sm_100a) windowed on-policy-distillation divergence library.
 *
 * The library evaluates, for every response position that lies inside its sequence's prefix
 * window, the teacher-student divergence over the full vocabulary, its gradient with respect to
 * the student logits, and the per-sequence / per-batch reductions that the prefix-versus-full
 * alignment audit consumes (ADWIN: Adaptive Windows for Horizon-Aware On-Policy Distillation).
 *
 * Notation: row r = (b,t); z = student_logits[b,t,:], u = teacher_logits[b,t,:], y = tokens[b,t];
 * p = softmax(z), q = softmax(u); W_b = window[b] (the training window L_t of Section 4.1, given
 * per sequence), R_b = rollout_len[b]; E_b = min(W_b, R_b, T) is the effective window.  Positions
 * are 0-based response positions; logits[b,t,:] is the distribution y[b,t] was drawn from (the
 * library never shifts).
 *
 * Pointer convention: every pointer is a DEVICE pointer owned by the caller unless its comment
 * says "host".  The library allocates nothing, frees nothing and never synchronises the stream:
 * all work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream).
 *
 * Errors: the int return value is an adwin_status_t detected on the host before anything is
 * launched (nothing is enqueued on error).  Conditions that only the device can see (array
 * contents) OR bits of adwin_dev_status_t into *dev_status; the kernels finish without faulting.
 */
#ifndef ADWIN_H_
#define ADWIN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ADWIN_OK = 0,
  ADWIN_ERR_NULL = 1,        /* a required pointer is NULL */
  ADWIN_ERR_SHAPE = 2,       /* B, T, V, ld, K out of range */
  ADWIN_ERR_ALIGN = 3,       /* a pointer is not aligned to its element type */
  ADWIN_ERR_DTYPE = 4,       /* unknown dtype / grad mode / flag */
  ADWIN_ERR_WINDOW = 5,      /* a host-visible W_b or R_b is negative, or R_b > T */
  ADWIN_ERR_WORKSPACE = 6,   /* workspace NULL, misaligned or smaller than adwin_workspace_bytes */
  ADWIN_ERR_CUDA = 7,        /* a CUDA runtime call failed (launch, attribute, copy) */
  ADWIN_ERR_UNSUPPORTED = 8  /* the requested combination is not implemented */
} adwin_status_t;

/* Bits OR-ed into *dev_status by the kernels. */
typedef enum {
  ADWIN_DEV_TOKEN_RANGE = 1, /* some processed tokens[b,t] outside [0,V): that row's logratio is NaN */
  ADWIN_DEV_NONFINITE = 2,   /* a processed row produced a non-finite log-sum-exp */
  ADWIN_DEV_TIMEOUT = 4,     /* a bounded on-chip wait ran out; outputs of this call are invalid */
  ADWIN_DEV_BOUNDS = 8,      /* an internal index check failed; outputs of this call are invalid */
  ADWIN_DEV_WINDOW = 16,     /* some W_b < 0, R_b < 0 or R_b > T; the value was clamped to [0,T] */
  ADWIN_DEV_WORKSPACE = 32   /* more processed positions than the workspace was sized for (the
                                max_rows bound of the fused LM-head call); nothing was computed */
} adwin_dev_status_t;

typedef enum { ADWIN_F32 = 0, ADWIN_BF16 = 1 } adwin_dtype_t;

/* Which gradient estimator the call evaluates (also decides what gsq is the squared norm of). */
typedef enum {
  ADWIN_GRAD_FULL_KL = 0, /* g_k = alpha p_k (log p_k - log q_k - KL): d/dz of the per-token reverse
                             KL(p||q), the full-vocabulary form of the OPD objective (Eq. 2) */
  ADWIN_GRAD_SAMPLED = 1  /* g_k = alpha c (1[k=y] - p_k): the gamma=0 token-local estimator
                             c_t * d log pi_theta(y_t) / dz (Eq. 4), c held constant */
} adwin_grad_mode_t;

enum {
  ADWIN_ZERO_TAIL = 1,     /* zero-fill gradient rows t >= E_b instead of leaving them untouched */
  ADWIN_RANGE_FULL = 2,    /* per-token scalars for every t < R_b (delayed full-rollout probe,
                              Section 4.2); the gradient is still written only for t < E_b */
  ADWIN_FORCE_GENERIC = 4, /* use the row-per-CTA streaming kernel for every row */
  ADWIN_FORCE_STAGED = 8   /* use the staged cluster kernel wherever the 16-byte layout allows,
                              also for calls without gradient (which by default go to the
                              streaming kernel: one sweep, nothing to keep on chip) */
};

/* Flags returned by adwin_probe_align in *flags_out. */
enum {
  ADWIN_ALIGN_DEGENERATE = 1,      /* some full-rollout squared norm was 0: that rho was set to 1 */
  ADWIN_ALIGN_NONE_ADMISSIBLE = 2  /* no candidate reached rho_star: L_next = largest candidate */
};

/* Library ABI version (bumped when a signature changes). */
int adwin_version(void);

/*
 * Diagnostic.  Every on-chip wait of the kernels (a consumer waiting for a bulk copy, a producer
 * for a free slot, the exchange between the CTAs of a cluster, the epilogue for an accumulator) is
 * bounded: when it runs out the kernel raises ADWIN_DEV_TIMEOUT, stops waiting anywhere, waits
 * for its own copies and MMAs in flight (those waits keep the full limit), frees its tensor
 * memory and returns; the outputs of that call are invalid, the context stays usable.  This sets
 * the limit of those handshake waits for the launches that follow, process-wide, in nanoseconds
 * (default 2 s; 0 restores the default).  A limit below 16 ns makes every wait that is not
 * satisfied at the moment it is reached run out, which is how the tests exercise the give-up path; there
 * is no other use for it.  The paper has no counterpart.
 */
void adwin_diag_set_wait_limit_ns(uint64_t ns);

/* Human-readable name of an adwin_status_t.  Host pointer to a static string. */
const char* adwin_status_string(int status);

/*
 * Bytes of device scratch that adwin_opd_kl_fwd_bwd wants for these shapes (the row map:
 * effective ranges and two sets of prefix sums, about 24 bytes per sequence).  Always > 0; the
 * buffer must be 256-byte aligned.  A buffer that holds only the first set (about two thirds of
 * this size) is still accepted: the call then runs an ADWIN_RANGE_FULL request with gradient as
 * one kernel instead of two, with the same results to within rounding.
 */
size_t adwin_workspace_bytes(int64_t B, int64_t T, int64_t V, int dtype, int flags);

/*
 * Windowed per-token OPD divergence, forward and backward, one pass over the logits.
 *
 * For every processed row (t < E_b; with ADWIN_RANGE_FULL: t < R_b) it computes, with fp32
 * accumulation,
 *   lse_s = log sum_k exp z_k, lse_t = log sum_k exp u_k        (log-softmax normalisers)
 *   kl[b,t]       = sum_k p_k (log p_k - log q_k)               reverse KL(p||q), per-token form of
 *                                                               the OPD objective (Eq. 2)
 *   logratio[b,t] = log p_y - log q_y                           step-wise cost c_t (Section 2.3);
 *                                                               the token reward is -c_t (App. A.1)
 *   gsq[b,t]      = sum_k g_k^2                                 squared norm of the row's gradient
 * and, when grad_student != NULL and t < E_b, writes g (see adwin_grad_mode_t, alpha = grad_scale)
 * to grad_student[b,t,:].  Rows past the window are skipped entirely: their logits are never read
 * and their gradient rows are left untouched (or zero-filled with ADWIN_ZERO_TAIL).  Per-token
 * outputs of rows that are not processed are written as 0.
 *
 * student_logits, teacher_logits : [B,T,V], element type `dtype`, row stride `ld` elements
 *                                  (row r = b*T+t starts at element r*ld; ld >= V)
 * tokens       : [B,T] int32            window : [B] int32
 * rollout_len  : [B] int32 or NULL (= T for every sequence)
 * grad_student : [B,T,V] of `grad_dtype`, row stride ld_grad, or NULL (no gradient is written;
 *                gsq is then accumulated in the same single sweep)
 * kl, logratio : [B,T] fp32, required.   gsq, lse_student, lse_teacher : [B,T] fp32 or NULL
 * workspace    : >= adwin_workspace_bytes(...) bytes, 256-byte aligned; contents undefined after
 * dev_status   : one int32 the caller zeroed; bits are OR-ed in
 *
 * Two kernels do the work, with identical results up to rounding order.  Rows whose gradient is
 * written go to the staged cluster kernel (two sweeps with the row kept on chip), which needs
 * 16-byte aligned logits / gradient base pointers, row strides that are multiples of 16 bytes and
 * V*sizeof(element) a multiple of 16.  Rows without gradient (a call with grad_student == NULL,
 * or the rows past the window of an ADWIN_RANGE_FULL call) and every other layout go to the
 * streaming kernel, one CTA per row.  ADWIN_FORCE_GENERIC / ADWIN_FORCE_STAGED override the choice.
 */
int adwin_opd_kl_fwd_bwd(const void* student_logits, const void* teacher_logits, int dtype,
                         int64_t B, int64_t T, int64_t V, int64_t ld, const int32_t* tokens,
                         const int32_t* window, const int32_t* rollout_len, float grad_scale,
                         int grad_mode, int flags, void* grad_student, int grad_dtype,
                         int64_t ld_grad, float* kl, float* logratio, float* gsq,
                         float* lse_student, float* lse_teacher, void* workspace,
                         size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * Windowed sums: the loss "on this prefix" that the synchronous update uses (Section 4.1).
 * seq_out[b] = { sum_{t<E_b} kl, sum_{t<E_b} logratio, sum_{t<E_b} gsq, E_b } and batch_out =
 * the same four summed over b, all in float64 with a fixed summation order (bitwise
 * reproducible).  gsq may be NULL (its sums are 0).  seq_out [B,4], batch_out [4]: device.
 */
int adwin_window_reduce(const float* kl, const float* logratio, const float* gsq,
                        const int32_t* window, const int32_t* rollout_len, int64_t B, int64_t T,
                        double* seq_out, double* batch_out, void* cuda_stream);

/*
 * Prefix-versus-full alignment audit on a returned probe batch (Section 4.2), in logit space.
 * Input: per-token scalars valid on t < R_b (a call with ADWIN_RANGE_FULL).  In logit space the
 * prefix gradient is the full-rollout gradient with rows t >= L zeroed, hence
 *   rho(L) = cos(u_probe, u^(L)) = sqrt(Q(L)/Q_full),   Q(L) = sum_{t < min(L,R_b)} gsq[b,t].
 * Slots j = 0..K-1 are the candidate lengths, slot K is each sequence's own W_b.
 *   seq_stats   [B,K+1,4] = { Q_b(L_j), sum kl, sum logratio over the same prefix, rho_b(L_j) }
 *   seq_full    [B,3]     = { Q_b_full, sum kl, sum logratio over t < R_b }
 *   batch_stats [K+1,5]   = { rho_micro, rho_macro, snr_micro, admissible (0/1), n_tokens }
 * rho_macro = mean over the B sequences of rho_b; rho_micro = the cosine after batch aggregation
 * (Figure 5); SNR = rho^2/(1-rho^2); admissible <=> rho_micro >= rho_star (threshold equation of Section 4.2, inclusive).
 * *L_next = the smallest admissible candidate (the scheduler rule of Section 4.2), or the largest
 * candidate with ADWIN_ALIGN_NONE_ADMISSIBLE.  A zero full norm gives rho = 1 and
 * ADWIN_ALIGN_DEGENERATE.
 * candidates : [K] int32 DEVICE pointer, or NULL for the paper's list {64,...,2048} (then K must
 *              be 0 or 6).  1 <= K <= 64.     rho_star <= 0 selects sqrt(2)/2.
 * All outputs are device pointers (float64 / int32), summed in a fixed order.
 */
int adwin_probe_align(const float* kl, const float* logratio, const float* gsq,
                      const int32_t* window, const int32_t* rollout_len, int64_t B, int64_t T,
                      const int32_t* candidates, int32_t K, double rho_star, double* seq_stats,
                      double* seq_full, double* batch_stats, int32_t* L_next, int32_t* flags_out,
                      void* cuda_stream);

/*
 * Discounted return-to-go of the per-token costs (Eq. 3; the derivation of the OPD gradient in the
 * appendix defines G_t^gamma):
 *     rtg[b,t] = sum_{t' = t}^{E_b - 1} gamma^(t'-t) * logratio[b,t']      for t < E_b,   0 elsewhere,
 * where E_b = min(W_b, R_b, T) is the end of the prefix window, or min(R_b, T) with
 * ADWIN_RANGE_FULL (the only flag accepted).  gamma = 0 returns the costs themselves (the
 * token-local estimator the paper trains with), gamma = 1 their suffix sums.
 * logratio, rtg : [B,T] float32 DEVICE pointers (rtg may not alias logratio); window, rollout_len
 * as in adwin_opd_kl_fwd_bwd (rollout_len may be NULL); out-of-range lengths are clamped to
 * [0,T] here (adwin_opd_kl_fwd_bwd reports them).  gamma outside [0,1] (or NaN) returns
 * ADWIN_ERR_SHAPE.  Sums are float64 in a fixed order; nothing is allocated or synchronised.
 */
int adwin_return_to_go(const float* logratio, const int32_t* window, const int32_t* rollout_len,
                       int64_t B, int64_t T, double gamma, int flags, float* rtg,
                       void* cuda_stream);

/*
 * adwin_opd_kl_fwd_bwd in ADWIN_GRAD_SAMPLED mode with a caller-supplied coefficient per
 * position in place of c_t:   g_k = grad_scale * row_coef[b,t] * (1[k = y] - p_k),
 * i.e. one term G_t * grad log pi_theta(y_t) of the future-coupled estimator (Eq. 3) in logit
 * space.  With gamma > 0 the coefficient of position t depends on later positions, so the caller
 * runs a read-only pass first (grad_student = NULL) for logratio, then adwin_return_to_go, then
 * this call.  row_coef : [B,T] float32 DEVICE pointer, read at the processed positions only.
 * All other arguments, outputs (kl, logratio, lse are those of the row; gsq is the squared norm
 * of the weighted gradient), layouts and errors are those of adwin_opd_kl_fwd_bwd.
 */
int adwin_opd_kl_fwd_bwd_weighted(const void* student_logits, const void* teacher_logits,
                                  int dtype, int64_t B, int64_t T, int64_t V, int64_t ld,
                                  const int32_t* tokens, const int32_t* window,
                                  const int32_t* rollout_len, const float* row_coef,
                                  float grad_scale, int flags, void* grad_student, int grad_dtype,
                                  int64_t ld_grad, float* kl, float* logratio, float* gsq,
                                  float* lse_student, float* lse_teacher, void* workspace,
                                  size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * Teacher-side drift along student rollouts (Section 3.1), one read of the teacher logits:
 *   entropy[b,t] = H[softmax(teacher_logits[b,t,:])] in nats; the teacher branching factor
 *                  (per-position perplexity) is BF = exp(entropy);
 *   rank[b,t]    = rank r of the sampled token tokens[b,t] under the teacher distribution,
 *                  1 + the number of vocabulary entries whose logit is strictly larger (equal
 *                  logits share the better rank); int32.
 * Positions t < R_b are processed (rollout_len NULL => T), the others get entropy 0 and rank 0.
 * Pointers, dtype, strides and dev_status as in adwin_opd_kl_fwd_bwd (no workspace is needed);
 * a token outside [0,V) gives rank 0 and ADWIN_DEV_TOKEN_RANGE, a non-finite entropy
 * ADWIN_DEV_NONFINITE, an invalid R_b is clamped and raises ADWIN_DEV_WINDOW.
 */
int adwin_teacher_drift(const void* teacher_logits, int dtype, int64_t B, int64_t T, int64_t V,
                        int64_t ld, const int32_t* tokens, const int32_t* rollout_len,
                        float* entropy, int32_t* rank, int32_t* dev_status, void* cuda_stream);

/*
 * The two curves of Section 3.1 over the B rollouts of a batch, per position t:
 *   worst_rank[b,t] = max_{t' <= t} rank[b,t']      [B,T] int32 (a rollout that has ended keeps
 *                     its value: it collects no further rejections);
 *   survival[j,t]   = (1/B) * #{b : worst_rank[b,t] <= ks[j]} = S_t^(k) for k = ks[j], the
 *                     fraction of rollouts with no top-k rejection through position t
 *                     (cumulative rejection is 1 - survival);   [K,T] float64, 0 <= K <= 64;
 *   bf_mean[t]      = mean of exp(entropy[b,t]) over the rollouts still running at t (t < R_b),
 *                     0 where none is;   [T] float64;        n_active[t] = their number, [T] int32.
 * entropy, rank: the outputs of adwin_teacher_drift.  ks: [K] int32 DEVICE pointer.  All pointers
 * are device pointers; sums run over the sequences in index order.
 */
int adwin_drift_curves(const float* entropy, const int32_t* rank, const int32_t* rollout_len,
                       int64_t B, int64_t T, const int32_t* ks, int32_t K, int32_t* worst_rank,
                       double* survival, double* bf_mean, int32_t* n_active, void* cuda_stream);

/*
 * The same divergence with both policies given as hidden states times an output embedding (the
 * form Eq. 2's policies have in a language model: pi = softmax(h W^T)), fused so that the logits
 * are never written to memory:
 *     z[b,t,:] = hidden_student[b,t,:] W_s^T,      u[b,t,:] = hidden_teacher[b,t,:] W_t^T,
 * then kl, logratio, gsq, lse_student, lse_teacher exactly as adwin_opd_kl_fwd_bwd defines them on
 * (z, u), and the gradients of the windowed loss with respect to the student's hidden states and
 * output embedding,
 *     grad_hidden[b,t,:] = G[b,t,:] W_s   for t < E_b,        grad_w = sum_{b, t < E_b} G[b,t,:]^T h_s[b,t,:],
 * where G is the logit gradient of the selected estimator (adwin_grad_mode_t, alpha = grad_scale).
 * grad_w is the student's LM-head block of the parameter-space gradient that Section 4.2's cosine
 * is defined on.  The products run on the tensor cores in bf16 with fp32 accumulation; G is
 * rounded to bf16 once before the two gradient products.
 *
 * hidden_student [B,T,d_s], w_student [V,d_s], hidden_teacher [B,T,d_t], w_teacher [V,d_t]:
 *                bf16, contiguous, 16-byte aligned; V, d_s, d_t multiples of 8
 * tokens, window, rollout_len, grad_scale, grad_mode: as in adwin_opd_kl_fwd_bwd
 * flags        : ADWIN_RANGE_FULL (per-token scalars for every t < R_b; gradients still from
 *                t < E_b only) and ADWIN_ZERO_TAIL (zero-fill grad_hidden rows t >= E_b; they are
 *                left untouched otherwise)
 * grad_hidden  : [B,T,d_s] of grad_hidden_dtype (ADWIN_F32 / ADWIN_BF16), or NULL
 * grad_w       : [V,d_s] fp32, overwritten (not accumulated into), or NULL
 * kl, logratio : [B,T] fp32, required.   gsq, lse_student, lse_teacher: [B,T] fp32 or NULL
 * max_rows     : an upper bound on the number of processed positions, sum_b E_b (sum_b R_b with
 *                ADWIN_RANGE_FULL), which sizes the workspace; <= 0 means B*T.  If the lengths on
 *                the device exceed it, ADWIN_DEV_WORKSPACE is raised and nothing is computed.
 * workspace    : >= adwin_lmhead_workspace_bytes(...) bytes, 1024-byte aligned; it holds compact
 *                copies of the processed hidden states, partial row statistics and, when a
 *                gradient is requested, G in bf16 (2 V bytes per processed position)
 * Errors as in adwin_opd_kl_fwd_bwd; shapes this path cannot take return ADWIN_ERR_UNSUPPORTED.
 */
size_t adwin_lmhead_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t d_s, int64_t d_t,
                                    int64_t max_rows, int flags, int with_grad);
int adwin_opd_kl_lmhead_fwd_bwd(const void* hidden_student, const void* w_student,
                                const void* hidden_teacher, const void* w_teacher, int64_t B,
                                int64_t T, int64_t V, int64_t d_s, int64_t d_t,
                                const int32_t* tokens, const int32_t* window,
                                const int32_t* rollout_len, float grad_scale, int grad_mode,
                                int flags, void* grad_hidden, int grad_hidden_dtype, float* grad_w,
                                float* kl, float* logratio, float* gsq, float* lse_student,
                                float* lse_teacher, int64_t max_rows, void* workspace,
                                size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * Prefix-versus-full alignment audit (Section 4.2) in the space of the student's LM-head weight,
 * on a returned probe batch given as hidden states.  For every candidate length L_j the prefix
 * gradient is dW^(L_j) = sum_b sum_{t < min(L_j, R_b)} G[b,t,:]^T h_s[b,t,:] and the full-horizon
 * reference dW^full the same sum over t < R_b (G = the logit gradient of the selected estimator,
 * every position of every rollout); then
 *   rho_w(L_j) = <dW^(L_j), dW^full> / (|dW^(L_j)| |dW^full|)     (the cosine after batch aggregation),
 * SNR = rho^2 / (1 - rho^2), admissible <=> rho_w >= rho_star, *L_next = the shortest admissible
 * candidate (the scheduler rule), or the largest one with ADWIN_ALIGN_NONE_ADMISSIBLE.  Unlike the
 * logit-space audit of adwin_probe_align this cosine sees the cancellation between positions and
 * samples (Figure 5) and can be negative.  A zero full norm gives rho = 1 and ADWIN_ALIGN_DEGENERATE,
 * a zero prefix norm rho = 0.
 *
 * hidden_*, w_*, tokens, rollout_len (NULL = T), grad_mode, max_rows (bound on sum_b R_b; <= 0 =
 * B*T), dev_status: as in adwin_opd_kl_lmhead_fwd_bwd.
 * candidates_host : HOST pointer to K strictly ascending multiples of 64 (they cut the positions
 *                   into bins of whole 64-row blocks), 1 <= K <= 16; NULL selects the paper's list
 *                   {64,...,2048} (then K must be 0 or 6).  rho_star <= 0 selects sqrt(2)/2.
 * kl, logratio, gsq : [B,T] fp32 per-token outputs over t < R_b (kl, logratio required).
 * batch_stats [K,4] = { rho_w, snr, admissible (0/1), n_tokens } float64; L_next, flags_out int32:
 *                   device pointers.
 * workspace       : >= adwin_lmhead_align_workspace_bytes(...) bytes, 1024-byte aligned: the
 *                   workspace of the fused pass plus K+1 fp32 matrices of the size of W_s.
 * The products run in bf16 with fp32 accumulation, G rounded to bf16 once; the cosines are formed
 * in float64 from the fp32 bin matrices in a fixed order.
 */
size_t adwin_lmhead_align_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t d_s,
                                          int64_t d_t, int64_t max_rows, int32_t K);
int adwin_lmhead_weight_align(const void* hidden_student, const void* w_student,
                              const void* hidden_teacher, const void* w_teacher, int64_t B,
                              int64_t T, int64_t V, int64_t d_s, int64_t d_t,
                              const int32_t* tokens, const int32_t* rollout_len,
                              const int32_t* candidates_host, int32_t K, double rho_star,
                              int grad_mode, float* kl, float* logratio, float* gsq,
                              double* batch_stats, int32_t* L_next, int32_t* flags_out,
                              int64_t max_rows, void* workspace, size_t workspace_bytes,
                              int32_t* dev_status, void* cuda_stream);

/*
 * The same pass for logits that live in HOST memory (pinned memory gives asynchronous copies).
 * Only the rows inside the processed range cross PCIe -- the window skip of Section 4.1 saves the
 * transfer as well as the arithmetic -- in stages of at most rows_per_stage rows of one sequence;
 * copies in, kernels and read-backs of neighbouring stages overlap on three streams (the kernels
 * run on cuda_stream; two internal copy streams are created on first use, per device).
 *
 * student_host, teacher_host, tokens_host, window_host, rollout_len_host, grad_host, kl_host,
 * logratio_host, gsq_host: HOST pointers with the shapes / strides of adwin_opd_kl_fwd_bwd.
 * The int32 length arrays are read during the call; everything else is read or written
 * asynchronously: synchronise cuda_stream before touching the outputs or reusing the inputs.
 * staging_dev : DEVICE scratch of >= adwin_host_staging_bytes(...) bytes, 256-byte aligned.
 * dev_status  : DEVICE int32, as in adwin_opd_kl_fwd_bwd.
 * Invalid lengths are host-visible here and return ADWIN_ERR_WINDOW before anything is enqueued.
 * The paper has no counterpart for this entry point: it is the end-to-end form of Section 4.1's
 * prefix evaluation for a trainer whose logits are produced on another device or host.
 */
size_t adwin_host_staging_bytes(int64_t rows_per_stage, int64_t V, int dtype, int grad_dtype,
                                int with_grad);
int adwin_opd_kl_fwd_bwd_host(const void* student_host, const void* teacher_host, int dtype,
                              int64_t B, int64_t T, int64_t V, int64_t ld,
                              const int32_t* tokens_host, const int32_t* window_host,
                              const int32_t* rollout_len_host, float grad_scale, int grad_mode,
                              int flags, void* grad_host, int grad_dtype, int64_t ld_grad,
                              float* kl_host, float* logratio_host, float* gsq_host,
                              void* staging_dev, size_t staging_bytes, int64_t rows_per_stage,
                              int32_t* dev_status, void* cuda_stream);

/*
 * adwin_opd_kl_fwd_bwd without a workspace argument and without any allocation.
 *
 * The paper has no counterpart for this entry point.  It is for callers that cannot supply
 * scratch memory and must not allocate: a trainer whose framework has claimed the whole GPU for
 * its own memory pool (a cudaMalloc there would fail, or take memory away from the pool), code
 * that runs where an allocation's implicit device-wide synchronisation is not acceptable, and
 * bindings from runtimes that expose no device allocator at all.  The row map that
 * adwin_opd_kl_fwd_bwd keeps in `workspace` is kept here in a fixed array inside the library
 * image (about 66 KB on every GPU that loads the library, held until the process exits).  The
 * call itself allocates and frees nothing, on the device or through any library.
 *
 * Arguments, outputs, rounding and error behaviour are those of adwin_opd_kl_fwd_bwd, with
 * `workspace` / `workspace_bytes` left out.  Differences:
 *   - B may be at most adwin_no_alloc_max_sequences() (4096); a larger batch returns
 *     ADWIN_ERR_WORKSPACE and enqueues nothing.  T and V are not limited by the array.
 *   - The array has room for the second set of prefix sums (the one that lets an
 *     ADWIN_RANGE_FULL call with gradient run as two kernels) only up to B = 2719; above that
 *     such a call runs as one kernel, with the same results to within rounding order.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current, as for every call).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call rewrites it completely before reading
 *     it, so nothing carries over from one call to the next, but two calls whose kernels can
 *     overlap on the GPU (different streams, no dependency between them) race on it and give
 *     undefined results: keep calls to this entry point ordered on one stream, or use
 *     adwin_opd_kl_fwd_bwd with separate workspaces.
 */
int64_t adwin_no_alloc_max_sequences(void);
int adwin_opd_kl_fwd_bwd_no_alloc(const void* student_logits, const void* teacher_logits,
                                  int dtype, int64_t B, int64_t T, int64_t V, int64_t ld,
                                  const int32_t* tokens, const int32_t* window,
                                  const int32_t* rollout_len, float grad_scale, int grad_mode,
                                  int flags, void* grad_student, int grad_dtype, int64_t ld_grad,
                                  float* kl, float* logratio, float* gsq, float* lse_student,
                                  float* lse_teacher, int32_t* dev_status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ADWIN_H_ */
