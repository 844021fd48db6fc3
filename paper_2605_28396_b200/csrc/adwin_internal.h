// Host-side declarations shared by the translation units of the library (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/adwin.h"

namespace adwin {

struct KlParams;

// Time limit of the kernels' handshake waits (consumer / producer / exchange / accumulator
// barriers), 2 s unless the diagnostic entry point shortened it.  The loops that wait for a
// kernel's own copies or MMAs in flight on its way out always keep the 2 s limit.
uint64_t handshake_wait_limit_ns();

// Workspace layout: [0,256) reserved counters; offsets (B+1) int64; range B int32; ewin B int32:
// `total` bytes, the part every call needs.  Optional extension up to `total_ext`: a second
// prefix-sum array over the effective windows, offsets_win (B+1) int64, which lets a call that
// wants scalars over the rollout and the gradient inside the window run as two kernels.
struct WorkspaceLayout {
  size_t off_offsets, off_range, off_ewin, total;
  size_t off_offsets_win, total_ext;
};
WorkspaceLayout workspace_layout(int64_t B);

cudaError_t launch_rowmap(const int32_t* window, const int32_t* rollout_len, int64_t B, int64_t T,
                          int flags, void* workspace, bool with_window_offsets, float* kl,
                          float* logratio, float* gsq, float* lse_s, float* lse_t, int32_t* status,
                          cudaStream_t s);

cudaError_t launch_zero_tail(const KlParams& p, int grad_dtype, cudaStream_t s);

cudaError_t launch_kl_generic(const KlParams& p, int dtype, int grad_dtype, bool vec, int sm_count,
                              cudaStream_t s);

// Staged cluster kernel.  Returns cudaErrorNotSupported when the shape does not fit its plan
// (the caller then falls back to the generic kernel).
cudaError_t launch_kl_staged(const KlParams& p, int dtype, int grad_dtype, int sm_count,
                             cudaStream_t s);

cudaError_t launch_window_reduce(const float* kl, const float* logratio, const float* gsq,
                                 const int32_t* window, const int32_t* rollout_len, int64_t B,
                                 int64_t T, double* seq_out, double* batch_out, cudaStream_t s);

cudaError_t launch_probe_align(const float* kl, const float* logratio, const float* gsq,
                               const int32_t* window, const int32_t* rollout_len, int64_t B,
                               int64_t T, const int32_t* candidates, int32_t K, double rho_star,
                               double* seq_stats, double* seq_full, double* batch_stats,
                               int32_t* L_next, int32_t* flags_out, cudaStream_t s);

cudaError_t launch_return_to_go(const float* logratio, const int32_t* window,
                                const int32_t* rollout_len, int64_t B, int64_t T, double gamma,
                                int flags, float* rtg, cudaStream_t s);

cudaError_t launch_teacher_drift(const void* teacher, int dtype, int64_t B, int64_t T, int64_t V,
                                 int64_t ld, const int32_t* tokens, const int32_t* rollout_len,
                                 float* entropy, int32_t* rank, int32_t* status, bool vec,
                                 int sm_count, cudaStream_t s);

cudaError_t launch_drift_curves(const float* entropy, const int32_t* rank,
                                const int32_t* rollout_len, int64_t B, int64_t T,
                                const int32_t* ks, int32_t K, int32_t* worst, double* survival,
                                double* bf_mean, int32_t* n_active, cudaStream_t s);

// Fused LM-head form (lmhead.cu).
void set_sweep_tile_columns(int bn);
void set_sweep_pair(int on);
size_t lmhead_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t ds, int64_t dt,
                              int64_t max_rows, bool want_grad, bool range_full);
cudaError_t launch_lmhead(const void* hs, const void* ws, const void* ht, const void* wt, int64_t B,
                          int64_t T, int64_t V, int64_t ds, int64_t dt, const int32_t* tokens,
                          const int32_t* window, const int32_t* rollout_len, float alpha, int mode,
                          int flags, void* dH, int dh_dtype, float* dW, float* kl, float* logratio,
                          float* gsq, float* lse_s, float* lse_t, void* workspace,
                          int64_t max_rows, int32_t* status, int sm_count, cudaStream_t s,
                          bool keep_G = false);
size_t lmhead_align_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t ds, int64_t dt,
                                    int64_t max_rows, int K);
cudaError_t launch_lmhead_weight_align(const void* hs, const void* ws, const void* ht,
                                       const void* wt, int64_t B, int64_t T, int64_t V, int64_t ds,
                                       int64_t dt, const int32_t* tokens,
                                       const int32_t* rollout_len, const int32_t* cand_host, int K,
                                       double rho_star, int mode, float* kl, float* logratio,
                                       float* gsq, double* batch_stats, int32_t* L_next,
                                       int32_t* flags_out, void* workspace, int64_t max_rows,
                                       int32_t* status, int sm_count, cudaStream_t s);
cudaError_t launch_tc_gemm(const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb,
                           bool b_mn, int64_t M, int64_t N, int64_t K, void* C, int64_t ldc,
                           bool c_bf16, const int32_t* m_tiles_dev, const int32_t* k_tiles_dev,
                           const int32_t* row_map, int32_t* status, int sm_count, cudaStream_t s,
                           const int32_t* k_list = nullptr, const int32_t* k_count_dev = nullptr);

}  // namespace adwin
