// extern "C" entry points: argument validation and kernel dispatch.  No allocation, no
// synchronisation; everything is enqueued on the caller's stream.
#include <atomic>
#include <mutex>

#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {

static std::atomic<uint64_t> g_handshake_limit_ns{2000000000ull};
uint64_t handshake_wait_limit_ns() { return g_handshake_limit_ns.load(); }

namespace {

constexpr int kKnownFlags =
    ADWIN_ZERO_TAIL | ADWIN_RANGE_FULL | ADWIN_FORCE_GENERIC | ADWIN_FORCE_STAGED;
constexpr int64_t kMaxB = int64_t(1) << 24;
constexpr int64_t kMaxT = int64_t(1) << 24;
constexpr int64_t kMaxV = int64_t(1) << 28;

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t elem_size(int dtype) { return dtype == ADWIN_F32 ? 4 : 2; }

int sm_count_of_current_device() {
  static std::mutex mu;
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
  std::lock_guard<std::mutex> lock(mu);
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      return -1;
    cached[dev] = n;
  }
  return cached[dev];
}

// Shared body of the two forward+backward entry points (row_coef is null for the plain one).
int opd_kl_fwd_bwd_impl(const void* student_logits, const void* teacher_logits, int dtype,
                        int64_t B, int64_t T, int64_t V, int64_t ld, const int32_t* tokens,
                        const int32_t* window, const int32_t* rollout_len, float grad_scale,
                        int grad_mode, int flags, void* grad_student, int grad_dtype,
                        int64_t ld_grad, float* kl, float* logratio, float* gsq,
                        float* lse_student, float* lse_teacher, void* workspace,
                        size_t workspace_bytes, int32_t* dev_status, void* cuda_stream,
                        const float* row_coef);

}  // namespace
}  // namespace adwin

using namespace adwin;

extern "C" {

int adwin_version(void) { return 2; }

void adwin_diag_set_wait_limit_ns(uint64_t ns) {
  g_handshake_limit_ns.store(ns == 0 ? 2000000000ull : ns);
}

const char* adwin_status_string(int status) {
  switch (status) {
    case ADWIN_OK: return "ADWIN_OK";
    case ADWIN_ERR_NULL: return "ADWIN_ERR_NULL: a required pointer is NULL";
    case ADWIN_ERR_SHAPE: return "ADWIN_ERR_SHAPE: a dimension or stride is out of range";
    case ADWIN_ERR_ALIGN: return "ADWIN_ERR_ALIGN: a pointer is not aligned to its element type";
    case ADWIN_ERR_DTYPE: return "ADWIN_ERR_DTYPE: unknown dtype, gradient mode or flag";
    case ADWIN_ERR_WINDOW: return "ADWIN_ERR_WINDOW: invalid window or rollout length";
    case ADWIN_ERR_WORKSPACE: return "ADWIN_ERR_WORKSPACE: workspace missing, misaligned or too small";
    case ADWIN_ERR_CUDA: return "ADWIN_ERR_CUDA: a CUDA runtime call failed";
    case ADWIN_ERR_UNSUPPORTED: return "ADWIN_ERR_UNSUPPORTED: combination not implemented";
    default: return "unknown adwin status";
  }
}

size_t adwin_workspace_bytes(int64_t B, int64_t T, int64_t V, int dtype, int flags) {
  (void)T; (void)V; (void)dtype; (void)flags;
  if (B < 0) B = 0;
  return workspace_layout(B).total_ext;
}

int adwin_opd_kl_fwd_bwd(const void* student_logits, const void* teacher_logits, int dtype,
                         int64_t B, int64_t T, int64_t V, int64_t ld, const int32_t* tokens,
                         const int32_t* window, const int32_t* rollout_len, float grad_scale,
                         int grad_mode, int flags, void* grad_student, int grad_dtype,
                         int64_t ld_grad, float* kl, float* logratio, float* gsq,
                         float* lse_student, float* lse_teacher, void* workspace,
                         size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  return opd_kl_fwd_bwd_impl(student_logits, teacher_logits, dtype, B, T, V, ld, tokens, window,
                             rollout_len, grad_scale, grad_mode, flags, grad_student, grad_dtype,
                             ld_grad, kl, logratio, gsq, lse_student, lse_teacher, workspace,
                             workspace_bytes, dev_status, cuda_stream, nullptr);
}

int adwin_opd_kl_fwd_bwd_weighted(const void* student_logits, const void* teacher_logits,
                                  int dtype, int64_t B, int64_t T, int64_t V, int64_t ld,
                                  const int32_t* tokens, const int32_t* window,
                                  const int32_t* rollout_len, const float* row_coef,
                                  float grad_scale, int flags, void* grad_student, int grad_dtype,
                                  int64_t ld_grad, float* kl, float* logratio, float* gsq,
                                  float* lse_student, float* lse_teacher, void* workspace,
                                  size_t workspace_bytes, int32_t* dev_status,
                                  void* cuda_stream) {
  if (B > 0 && T > 0 && !row_coef) return ADWIN_ERR_NULL;
  if (!aligned(row_coef, 4)) return ADWIN_ERR_ALIGN;
  return opd_kl_fwd_bwd_impl(student_logits, teacher_logits, dtype, B, T, V, ld, tokens, window,
                             rollout_len, grad_scale, ADWIN_GRAD_SAMPLED, flags, grad_student,
                             grad_dtype, ld_grad, kl, logratio, gsq, lse_student, lse_teacher,
                             workspace, workspace_bytes, dev_status, cuda_stream, row_coef);
}

int adwin_return_to_go(const float* logratio, const int32_t* window, const int32_t* rollout_len,
                       int64_t B, int64_t T, double gamma, int flags, float* rtg,
                       void* cuda_stream) {
  if (flags & ~ADWIN_RANGE_FULL) return ADWIN_ERR_DTYPE;
  if (B < 0 || T < 0 || B > kMaxB || T > kMaxT) return ADWIN_ERR_SHAPE;
  if (!(gamma >= 0.0 && gamma <= 1.0)) return ADWIN_ERR_SHAPE;
  if (B == 0 || T == 0) return ADWIN_OK;
  if (!logratio || !window || !rtg) return ADWIN_ERR_NULL;
  if (!aligned(logratio, 4) || !aligned(window, 4) || !aligned(rollout_len, 4) || !aligned(rtg, 4))
    return ADWIN_ERR_ALIGN;
  if (launch_return_to_go(logratio, window, rollout_len, B, T, gamma, flags, rtg,
                          static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

int adwin_teacher_drift(const void* teacher_logits, int dtype, int64_t B, int64_t T, int64_t V,
                        int64_t ld, const int32_t* tokens, const int32_t* rollout_len,
                        float* entropy, int32_t* rank, int32_t* dev_status, void* cuda_stream) {
  if (dtype != ADWIN_F32 && dtype != ADWIN_BF16) return ADWIN_ERR_DTYPE;
  if (B < 0 || T < 0 || B > kMaxB || T > kMaxT || V < 1 || V > kMaxV || ld < V)
    return ADWIN_ERR_SHAPE;
  if (!dev_status) return ADWIN_ERR_NULL;
  if (B == 0 || T == 0) return ADWIN_OK;
  if (!teacher_logits || !tokens || !entropy || !rank) return ADWIN_ERR_NULL;
  const size_t es = elem_size(dtype);
  if (!aligned(teacher_logits, es) || !aligned(tokens, 4) || !aligned(rollout_len, 4) ||
      !aligned(entropy, 4) || !aligned(rank, 4) || !aligned(dev_status, 4))
    return ADWIN_ERR_ALIGN;
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return ADWIN_ERR_CUDA;
  const bool vec16 = aligned(teacher_logits, 16) && (ld * es) % 16 == 0 && (V * es) % 16 == 0;
  if (launch_teacher_drift(teacher_logits, dtype, B, T, V, ld, tokens, rollout_len, entropy, rank,
                           dev_status, vec16, sms,
                           static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

int adwin_drift_curves(const float* entropy, const int32_t* rank, const int32_t* rollout_len,
                       int64_t B, int64_t T, const int32_t* ks, int32_t K, int32_t* worst_rank,
                       double* survival, double* bf_mean, int32_t* n_active, void* cuda_stream) {
  if (B < 0 || T < 0 || B > kMaxB || T > kMaxT || K < 0 || K > 64) return ADWIN_ERR_SHAPE;
  if (B == 0 || T == 0) return ADWIN_OK;
  if (!entropy || !rank || !worst_rank || !bf_mean || !n_active) return ADWIN_ERR_NULL;
  if (K > 0 && (!ks || !survival)) return ADWIN_ERR_NULL;
  if (!aligned(entropy, 4) || !aligned(rank, 4) || !aligned(rollout_len, 4) || !aligned(ks, 4) ||
      !aligned(worst_rank, 4) || !aligned(survival, 8) || !aligned(bf_mean, 8) ||
      !aligned(n_active, 4))
    return ADWIN_ERR_ALIGN;
  if (launch_drift_curves(entropy, rank, rollout_len, B, T, ks, K, worst_rank, survival, bf_mean,
                          n_active, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

}  // extern "C"

namespace adwin {
namespace {

int opd_kl_fwd_bwd_impl(const void* student_logits, const void* teacher_logits, int dtype,
                        int64_t B, int64_t T, int64_t V, int64_t ld, const int32_t* tokens,
                        const int32_t* window, const int32_t* rollout_len, float grad_scale,
                        int grad_mode, int flags, void* grad_student, int grad_dtype,
                        int64_t ld_grad, float* kl, float* logratio, float* gsq,
                        float* lse_student, float* lse_teacher, void* workspace,
                        size_t workspace_bytes, int32_t* dev_status, void* cuda_stream,
                        const float* row_coef) {
  if (dtype != ADWIN_F32 && dtype != ADWIN_BF16) return ADWIN_ERR_DTYPE;
  if (grad_mode != ADWIN_GRAD_FULL_KL && grad_mode != ADWIN_GRAD_SAMPLED) return ADWIN_ERR_DTYPE;
  if (flags & ~kKnownFlags) return ADWIN_ERR_DTYPE;
  if (grad_student && grad_dtype != ADWIN_F32 && grad_dtype != ADWIN_BF16) return ADWIN_ERR_DTYPE;
  if (B < 0 || T < 0 || B > kMaxB || T > kMaxT || V < 1 || V > kMaxV || ld < V)
    return ADWIN_ERR_SHAPE;
  if (grad_student && ld_grad < V) return ADWIN_ERR_SHAPE;
  if (!dev_status) return ADWIN_ERR_NULL;
  if (B == 0 || T == 0) return ADWIN_OK;
  if (!student_logits || !teacher_logits || !tokens || !window || !kl || !logratio)
    return ADWIN_ERR_NULL;
  const size_t es = elem_size(dtype);
  if (!aligned(student_logits, es) || !aligned(teacher_logits, es) || !aligned(tokens, 4) ||
      !aligned(window, 4) || !aligned(rollout_len, 4) || !aligned(kl, 4) ||
      !aligned(logratio, 4) || !aligned(gsq, 4) || !aligned(lse_student, 4) ||
      !aligned(lse_teacher, 4) || !aligned(dev_status, 4))
    return ADWIN_ERR_ALIGN;
  if (grad_student && !aligned(grad_student, elem_size(grad_dtype))) return ADWIN_ERR_ALIGN;
  if (!workspace || !aligned(workspace, 256) ||
      workspace_bytes < workspace_layout(B).total)
    return ADWIN_ERR_WORKSPACE;
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return ADWIN_ERR_CUDA;

  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const WorkspaceLayout wl = workspace_layout(B);
  char* wbase = static_cast<char*>(workspace);

  KlParams p;
  p.student = student_logits;
  p.teacher = teacher_logits;
  p.B = B; p.T = T; p.V = V; p.ld = ld;
  p.tokens = tokens;
  p.alpha = grad_scale;
  p.mode = grad_mode;
  p.flags = flags;
  p.grad = grad_student;
  p.ld_grad = grad_student ? ld_grad : 0;
  p.kl = kl; p.logratio = logratio; p.gsq = gsq; p.lse_s = lse_student; p.lse_t = lse_teacher;
  p.status = dev_status;
  p.offsets = reinterpret_cast<const int64_t*>(wbase + wl.off_offsets);
  p.range = reinterpret_cast<const int32_t*>(wbase + wl.off_range);
  p.ewin = reinterpret_cast<const int32_t*>(wbase + wl.off_ewin);
  p.row_coef = row_coef;
  p.skip_below = nullptr;

  // 16-byte layout test shared by the vectorised streaming path and the staged kernel.
  const int gd = grad_student ? grad_dtype : dtype;
  bool vec16 = aligned(student_logits, 16) && aligned(teacher_logits, 16) &&
               (ld * es) % 16 == 0 && (V * es) % 16 == 0;
  if (grad_student)
    vec16 = vec16 && aligned(grad_student, 16) && (ld_grad * elem_size(gd)) % 16 == 0 &&
            (V * elem_size(gd)) % 16 == 0;
  // Scalars over the whole rollout with the gradient inside the window: the window rows need the
  // staged kernel's two sweeps, the rows past the window are a single read, which the streaming
  // kernel does faster.  With the extended workspace the call runs them as two launches.
  const bool split = vec16 && grad_student && (flags & ADWIN_RANGE_FULL) &&
                     !(flags & (ADWIN_FORCE_GENERIC | ADWIN_FORCE_STAGED)) &&
                     workspace_bytes >= wl.total_ext;

  if (launch_rowmap(window, rollout_len, B, T, flags, workspace, split, kl, logratio, gsq,
                    lse_student, lse_teacher, dev_status, s) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  if ((flags & ADWIN_ZERO_TAIL) && grad_student) {
    if (launch_zero_tail(p, grad_dtype, s) != cudaSuccess) return ADWIN_ERR_CUDA;
  }

  if (split) {
    KlParams pw = p;          // window rows: the compact list built from the effective windows
    pw.offsets = reinterpret_cast<const int64_t*>(wbase + wl.off_offsets_win);
    pw.range = p.ewin;
    const cudaError_t e = launch_kl_staged(pw, dtype, gd, sms, s);
    if (e == cudaSuccess) {
      KlParams pr = p;        // the rest of every rollout, without gradient
      pr.grad = nullptr;
      pr.ld_grad = 0;
      pr.skip_below = p.ewin;
      if (launch_kl_generic(pr, dtype, dtype, true, sms, s) != cudaSuccess) return ADWIN_ERR_CUDA;
      return ADWIN_OK;
    }
    if (e != cudaErrorNotSupported) return ADWIN_ERR_CUDA;
  }
  // Rows whose gradient is written need two sweeps with the row kept on chip in between: the
  // staged cluster kernel.  A call without gradient is a single read of every row, which the
  // row-per-CTA streaming kernel does faster (90 % against 74 % of the copy bandwidth, measured).
  const bool want_staged = (flags & ADWIN_FORCE_STAGED) || grad_student != nullptr;
  if (vec16 && want_staged && !(flags & ADWIN_FORCE_GENERIC)) {
    const cudaError_t e = launch_kl_staged(p, dtype, gd, sms, s);
    if (e == cudaSuccess) return ADWIN_OK;
    if (e != cudaErrorNotSupported) return ADWIN_ERR_CUDA;
  }
  if (launch_kl_generic(p, dtype, gd, vec16, sms, s) != cudaSuccess) return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

}  // namespace
}  // namespace adwin

extern "C" {

int adwin_window_reduce(const float* kl, const float* logratio, const float* gsq,
                        const int32_t* window, const int32_t* rollout_len, int64_t B, int64_t T,
                        double* seq_out, double* batch_out, void* cuda_stream) {
  if (B < 0 || T < 0 || B > kMaxB || T > kMaxT) return ADWIN_ERR_SHAPE;
  if (!batch_out) return ADWIN_ERR_NULL;
  if (B > 0 && (!kl || !logratio || !window || !seq_out)) return ADWIN_ERR_NULL;
  if (!aligned(kl, 4) || !aligned(logratio, 4) || !aligned(gsq, 4) || !aligned(window, 4) ||
      !aligned(rollout_len, 4) || !aligned(seq_out, 8) || !aligned(batch_out, 8))
    return ADWIN_ERR_ALIGN;
  if (launch_window_reduce(kl, logratio, gsq, window, rollout_len, B, T, seq_out, batch_out,
                           static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

int adwin_probe_align(const float* kl, const float* logratio, const float* gsq,
                      const int32_t* window, const int32_t* rollout_len, int64_t B, int64_t T,
                      const int32_t* candidates, int32_t K, double rho_star, double* seq_stats,
                      double* seq_full, double* batch_stats, int32_t* L_next, int32_t* flags_out,
                      void* cuda_stream) {
  if (B < 0 || T < 0 || B > kMaxB || T > kMaxT) return ADWIN_ERR_SHAPE;
  if (!candidates) {
    if (K != 0 && K != 6) return ADWIN_ERR_SHAPE;
    K = 6;
  }
  if (K < 1 || K > 64) return ADWIN_ERR_SHAPE;
  if (!batch_stats || !L_next || !flags_out) return ADWIN_ERR_NULL;
  if (B > 0 && (!kl || !logratio || !gsq || !window || !seq_stats || !seq_full))
    return ADWIN_ERR_NULL;
  if (!aligned(kl, 4) || !aligned(logratio, 4) || !aligned(gsq, 4) || !aligned(window, 4) ||
      !aligned(rollout_len, 4) || !aligned(candidates, 4) || !aligned(seq_stats, 8) ||
      !aligned(seq_full, 8) || !aligned(batch_stats, 8) || !aligned(L_next, 4) ||
      !aligned(flags_out, 4))
    return ADWIN_ERR_ALIGN;
  if (!(rho_star > 0.0)) rho_star = 0.70710678118654752440;  // sqrt(2)/2
  if (launch_probe_align(kl, logratio, gsq, window, rollout_len, B, T, candidates, K, rho_star,
                         seq_stats, seq_full, batch_stats, L_next, flags_out,
                         static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

size_t adwin_lmhead_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t d_s, int64_t d_t,
                                    int64_t max_rows, int flags, int with_grad) {
  if (B < 0) B = 0;
  if (T < 0) T = 0;
  if (V < 1) V = 1;
  if (d_s < 1) d_s = 1;
  if (d_t < 1) d_t = 1;
  return lmhead_workspace_bytes(B, T, V, d_s, d_t, max_rows, with_grad != 0,
                                (flags & ADWIN_RANGE_FULL) != 0);
}

int adwin_opd_kl_lmhead_fwd_bwd(const void* hidden_student, const void* w_student,
                                const void* hidden_teacher, const void* w_teacher, int64_t B,
                                int64_t T, int64_t V, int64_t d_s, int64_t d_t,
                                const int32_t* tokens, const int32_t* window,
                                const int32_t* rollout_len, float grad_scale, int grad_mode,
                                int flags, void* grad_hidden, int grad_hidden_dtype, float* grad_w,
                                float* kl, float* logratio, float* gsq, float* lse_student,
                                float* lse_teacher, int64_t max_rows, void* workspace,
                                size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  if (grad_mode != ADWIN_GRAD_FULL_KL && grad_mode != ADWIN_GRAD_SAMPLED) return ADWIN_ERR_DTYPE;
  if (flags & ~(ADWIN_RANGE_FULL | ADWIN_ZERO_TAIL)) return ADWIN_ERR_DTYPE;
  if (grad_hidden && grad_hidden_dtype != ADWIN_F32 && grad_hidden_dtype != ADWIN_BF16)
    return ADWIN_ERR_DTYPE;
  if (B < 0 || T < 0 || B > 65536 || T > kMaxT || V < 1 || V > kMaxV || d_s < 1 || d_t < 1 ||
      d_s > (int64_t(1) << 20) || d_t > (int64_t(1) << 20))
    return ADWIN_ERR_SHAPE;
  if (!dev_status) return ADWIN_ERR_NULL;
  if (B == 0 || T == 0) return ADWIN_OK;
  if (!hidden_student || !w_student || !hidden_teacher || !w_teacher || !tokens || !window ||
      !kl || !logratio)
    return ADWIN_ERR_NULL;
  if ((V % 8) || (d_s % 8) || (d_t % 8) || B * T > (int64_t(1) << 30)) return ADWIN_ERR_UNSUPPORTED;
  if (!aligned(hidden_student, 16) || !aligned(w_student, 16) || !aligned(hidden_teacher, 16) ||
      !aligned(w_teacher, 16) || !aligned(grad_hidden, 16) || !aligned(grad_w, 16) ||
      !aligned(tokens, 4) || !aligned(window, 4) || !aligned(rollout_len, 4) || !aligned(kl, 4) ||
      !aligned(logratio, 4) || !aligned(gsq, 4) || !aligned(lse_student, 4) ||
      !aligned(lse_teacher, 4) || !aligned(dev_status, 4))
    return ADWIN_ERR_ALIGN;
  const bool want_grad = grad_hidden || grad_w;
  if (!workspace || !aligned(workspace, 1024) ||
      workspace_bytes < lmhead_workspace_bytes(B, T, V, d_s, d_t, max_rows, want_grad,
                                               (flags & ADWIN_RANGE_FULL) != 0))
    return ADWIN_ERR_WORKSPACE;
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return ADWIN_ERR_CUDA;
  if (launch_lmhead(hidden_student, w_student, hidden_teacher, w_teacher, B, T, V, d_s, d_t, tokens,
                    window, rollout_len, grad_scale, grad_mode, flags, grad_hidden,
                    grad_hidden_dtype, grad_w, kl, logratio, gsq, lse_student, lse_teacher,
                    workspace, max_rows, dev_status, sms,
                    static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

size_t adwin_lmhead_align_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t d_s,
                                          int64_t d_t, int64_t max_rows, int32_t K) {
  if (B < 0) B = 0;
  if (T < 0) T = 0;
  if (V < 1) V = 1;
  if (d_s < 1) d_s = 1;
  if (d_t < 1) d_t = 1;
  if (K < 1) K = 6;
  if (K > 16) K = 16;
  return lmhead_align_workspace_bytes(B, T, V, d_s, d_t, max_rows, K);
}

int adwin_lmhead_weight_align(const void* hidden_student, const void* w_student,
                              const void* hidden_teacher, const void* w_teacher, int64_t B,
                              int64_t T, int64_t V, int64_t d_s, int64_t d_t,
                              const int32_t* tokens, const int32_t* rollout_len,
                              const int32_t* candidates_host, int32_t K, double rho_star,
                              int grad_mode, float* kl, float* logratio, float* gsq,
                              double* batch_stats, int32_t* L_next, int32_t* flags_out,
                              int64_t max_rows, void* workspace, size_t workspace_bytes,
                              int32_t* dev_status, void* cuda_stream) {
  static const int32_t kPaperList[6] = {64, 128, 256, 512, 1024, 2048};
  if (grad_mode != ADWIN_GRAD_FULL_KL && grad_mode != ADWIN_GRAD_SAMPLED) return ADWIN_ERR_DTYPE;
  if (!candidates_host) {
    if (K != 0 && K != 6) return ADWIN_ERR_SHAPE;
    candidates_host = kPaperList;
    K = 6;
  }
  if (K < 1 || K > 16) return ADWIN_ERR_SHAPE;
  for (int i = 0; i < K; ++i) {
    if (candidates_host[i] <= 0 || candidates_host[i] % 64 != 0) return ADWIN_ERR_SHAPE;
    if (i > 0 && candidates_host[i] <= candidates_host[i - 1]) return ADWIN_ERR_SHAPE;
  }
  if (B < 0 || T < 0 || B > 65536 || T > kMaxT || V < 1 || V > kMaxV || d_s < 1 || d_t < 1 ||
      d_s > (int64_t(1) << 20) || d_t > (int64_t(1) << 20))
    return ADWIN_ERR_SHAPE;
  if (!dev_status || !batch_stats || !L_next || !flags_out) return ADWIN_ERR_NULL;
  if (B > 0 && T > 0 &&
      (!hidden_student || !w_student || !hidden_teacher || !w_teacher || !tokens || !kl || !logratio))
    return ADWIN_ERR_NULL;
  if ((V % 8) || (d_s % 8) || (d_t % 8) || B * T > (int64_t(1) << 30)) return ADWIN_ERR_UNSUPPORTED;
  if (!aligned(hidden_student, 16) || !aligned(w_student, 16) || !aligned(hidden_teacher, 16) ||
      !aligned(w_teacher, 16) || !aligned(tokens, 4) || !aligned(rollout_len, 4) ||
      !aligned(kl, 4) || !aligned(logratio, 4) || !aligned(gsq, 4) || !aligned(batch_stats, 8) ||
      !aligned(L_next, 4) || !aligned(flags_out, 4) || !aligned(dev_status, 4))
    return ADWIN_ERR_ALIGN;
  if (!workspace || !aligned(workspace, 1024) ||
      workspace_bytes < lmhead_align_workspace_bytes(B, T, V, d_s, d_t, max_rows, K))
    return ADWIN_ERR_WORKSPACE;
  if (!(rho_star > 0.0)) rho_star = 0.70710678118654752440;  // sqrt(2)/2
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return ADWIN_ERR_CUDA;
  if (launch_lmhead_weight_align(hidden_student, w_student, hidden_teacher, w_teacher, B, T, V, d_s,
                                 d_t, tokens, rollout_len, candidates_host, K, rho_star, grad_mode,
                                 kl, logratio, gsq, batch_stats, L_next, flags_out, workspace,
                                 max_rows, dev_status, sms,
                                 static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return ADWIN_ERR_CUDA;
  return ADWIN_OK;
}

#ifdef ADWIN_DEV_EXPORTS
void adwin_dev_set_sweep_bn(int bn) { set_sweep_tile_columns(bn); }
void adwin_dev_set_sweep_pair(int on) { set_sweep_pair(on); }
// Development build only: the tensor-core GEMM on its own, C = A B (bf16 in, fp32 or bf16 out).
int adwin_dev_gemm(const void* A, int64_t lda, int a_mn, const void* Bm, int64_t ldb, int b_mn,
                   int64_t M, int64_t N, int64_t K, void* C, int64_t ldc, int c_bf16,
                   int32_t* dev_status, void* cuda_stream) {
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return ADWIN_ERR_CUDA;
  return launch_tc_gemm(A, lda, a_mn != 0, Bm, ldb, b_mn != 0, M, N, K, C, ldc, c_bf16 != 0,
                        nullptr, nullptr, nullptr, dev_status, sms,
                        static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? ADWIN_OK
             : ADWIN_ERR_CUDA;
}
#endif

}  // extern "C"
