// Per-sequence / per-batch reductions over the [B,T] per-token scalars.
//
// adwin_window_reduce: the loss on the prefix window that the synchronous update uses.
// adwin_probe_align:   the prefix-versus-full alignment audit on a returned probe batch: in logit
//   space the prefix gradient is the full gradient with rows t >= L zeroed, so
//   rho(L) = sqrt(Q(L)/Q_full) with Q = sums of per-token squared gradient norms;
//   SNR = rho^2/(1-rho^2); admissible when rho >= rho_star; L_next = shortest admissible length.
// All sums are float64 in a fixed order (strided per thread, then a fixed tree), so results are
// bitwise reproducible.  These kernels touch O(B*T*K) floats: negligible next to the logit sweep.
#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {

constexpr int kRedThreads = 256;

// Fixed-order CTA sum of up to 3 doubles per thread; result valid in every thread.
__device__ __forceinline__ void block_sum3(double (&v)[3], double (*sm)[kRedThreads]) {
  const int tid = threadIdx.x;
#pragma unroll
  for (int i = 0; i < 3; ++i) sm[i][tid] = v[i];
  __syncthreads();
  for (int o = kRedThreads / 2; o > 0; o >>= 1) {
    if (tid < o) {
#pragma unroll
      for (int i = 0; i < 3; ++i) sm[i][tid] += sm[i][tid + o];
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 3; ++i) v[i] = sm[i][0];
  __syncthreads();
}

__device__ __forceinline__ int effective_len(const int32_t* rollout_len, int64_t b, int64_t T) {
  int64_t r = rollout_len ? rollout_len[b] : T;
  r = r < 0 ? 0 : (r > T ? T : r);
  return (int)r;
}

// Sums of (gsq, kl, logratio) over t < n of sequence b.
__device__ __forceinline__ void prefix_sums(const float* kl, const float* c, const float* gsq,
                                            int64_t b, int64_t T, int n, double (&out)[3],
                                            double (*sm)[kRedThreads]) {
  double v[3] = {0.0, 0.0, 0.0};
  for (int t = threadIdx.x; t < n; t += kRedThreads) {
    const int64_t i = b * T + t;
    v[0] += gsq ? (double)gsq[i] : 0.0;
    v[1] += (double)kl[i];
    v[2] += (double)c[i];
  }
  block_sum3(v, sm);
  out[0] = v[0];
  out[1] = v[1];
  out[2] = v[2];
}

__global__ void __launch_bounds__(kRedThreads) window_reduce_seq_kernel(
    const float* kl, const float* c, const float* gsq, const int32_t* window,
    const int32_t* rollout_len, int64_t B, int64_t T, double* seq_out) {
  __shared__ double sm[3][kRedThreads];
  for (int64_t b = blockIdx.x; b < B; b += gridDim.x) {
    const int R = effective_len(rollout_len, b, T);
    const int W = window[b] < 0 ? 0 : window[b];
    const int E = W < R ? W : R;
    double s[3];
    prefix_sums(kl, c, gsq, b, T, E, s, sm);
    if (threadIdx.x == 0) {
      seq_out[b * 4 + 0] = s[1];
      seq_out[b * 4 + 1] = s[2];
      seq_out[b * 4 + 2] = s[0];
      seq_out[b * 4 + 3] = (double)E;
    }
  }
}

// batch_out[i] = sum_b seq_out[b][i], i < 4, sequential in b (one thread per column).
__global__ void window_reduce_batch_kernel(const double* seq_out, int64_t B, double* batch_out) {
  const int i = threadIdx.x;
  if (i < 4) {
    double s = 0.0;
    for (int64_t b = 0; b < B; ++b) s += seq_out[b * 4 + i];
    batch_out[i] = s;
  }
}

cudaError_t launch_window_reduce(const float* kl, const float* logratio, const float* gsq,
                                 const int32_t* window, const int32_t* rollout_len, int64_t B,
                                 int64_t T, double* seq_out, double* batch_out, cudaStream_t s) {
  if (B > 0) {
    const int grid = (int)(B < 4096 ? B : 4096);
    window_reduce_seq_kernel<<<grid, kRedThreads, 0, s>>>(kl, logratio, gsq, window, rollout_len,
                                                          B, T, seq_out);
  }
  window_reduce_batch_kernel<<<1, 32, 0, s>>>(seq_out, B, batch_out);
  return cudaGetLastError();
}

__constant__ int32_t kDefaultCandidates[6] = {64, 128, 256, 512, 1024, 2048};

__device__ __forceinline__ int candidate_len(const int32_t* candidates, int j) {
  return candidates ? candidates[j] : kDefaultCandidates[j];
}

__global__ void __launch_bounds__(kRedThreads) probe_align_seq_kernel(
    const float* kl, const float* c, const float* gsq, const int32_t* window,
    const int32_t* rollout_len, int64_t B, int64_t T, const int32_t* candidates, int K,
    double* seq_stats, double* seq_full, int32_t* flags_out) {
  __shared__ double sm[3][kRedThreads];
  for (int64_t b = blockIdx.x; b < B; b += gridDim.x) {
    const int R = effective_len(rollout_len, b, T);
    double full[3];
    prefix_sums(kl, c, gsq, b, T, R, full, sm);
    if (threadIdx.x == 0) {
      seq_full[b * 3 + 0] = full[0];
      seq_full[b * 3 + 1] = full[1];
      seq_full[b * 3 + 2] = full[2];
      if (!(full[0] > 0.0)) atomicOr(flags_out, ADWIN_ALIGN_DEGENERATE);
    }
    for (int j = 0; j <= K; ++j) {
      int L = (j < K) ? candidate_len(candidates, j) : window[b];
      L = L < 0 ? 0 : L;
      const int n = L < R ? L : R;
      double s[3];
      prefix_sums(kl, c, gsq, b, T, n, s, sm);
      if (threadIdx.x == 0) {
        double* o = seq_stats + ((size_t)b * (K + 1) + j) * 4;
        o[0] = s[0];
        o[1] = s[1];
        o[2] = s[2];
        o[3] = (full[0] > 0.0) ? sqrt(s[0] / full[0]) : 1.0;
      }
    }
  }
}

// One thread per slot j: sequential sums over b, then rho / SNR / admissibility; thread 0 picks
// L_next after a barrier.
__global__ void probe_align_batch_kernel(const double* seq_stats, const double* seq_full,
                                         const int32_t* window, const int32_t* rollout_len,
                                         int64_t B, int64_t T, const int32_t* candidates, int K,
                                         double rho_star, double* batch_stats, int32_t* L_next,
                                         int32_t* flags_out) {
  __shared__ int admissible[65];
  const int j = threadIdx.x;
  if (j <= K) {
    double qp = 0.0, qf = 0.0, macro = 0.0, ntok = 0.0;
    for (int64_t b = 0; b < B; ++b) {
      const double* o = seq_stats + ((size_t)b * (K + 1) + j) * 4;
      qp += o[0];
      qf += seq_full[b * 3 + 0];
      macro += o[3];
      const int R = effective_len(rollout_len, b, T);
      int L = (j < K) ? candidate_len(candidates, j) : window[b];
      L = L < 0 ? 0 : L;
      ntok += (double)(L < R ? L : R);
    }
    double micro;
    if (qf > 0.0) {
      micro = sqrt(qp / qf);
    } else {
      micro = 1.0;
      atomicOr(flags_out, ADWIN_ALIGN_DEGENERATE);
    }
    const double r2 = micro * micro;
    double* o = batch_stats + j * 5;
    o[0] = micro;
    o[1] = (B > 0) ? macro / (double)B : 1.0;
    o[2] = (r2 < 1.0) ? r2 / (1.0 - r2) : (double)INFINITY;
    o[3] = (micro >= rho_star) ? 1.0 : 0.0;
    o[4] = ntok;
    admissible[j] = (micro >= rho_star) ? 1 : 0;
  }
  __syncthreads();
  if (j == 0) {
    int best = -1, largest = -1;
    for (int i = 0; i < K; ++i) {
      const int L = candidate_len(candidates, i);
      if (L > largest) largest = L;
      if (admissible[i] && (best < 0 || L < best)) best = L;
    }
    if (best < 0) {
      best = largest;
      atomicOr(flags_out, ADWIN_ALIGN_NONE_ADMISSIBLE);
    }
    *L_next = best;
  }
}

__global__ void clear_flag_kernel(int32_t* flags_out) { *flags_out = 0; }

cudaError_t launch_probe_align(const float* kl, const float* logratio, const float* gsq,
                               const int32_t* window, const int32_t* rollout_len, int64_t B,
                               int64_t T, const int32_t* candidates, int32_t K, double rho_star,
                               double* seq_stats, double* seq_full, double* batch_stats,
                               int32_t* L_next, int32_t* flags_out, cudaStream_t s) {
  clear_flag_kernel<<<1, 1, 0, s>>>(flags_out);
  if (B > 0) {
    const int grid = (int)(B < 4096 ? B : 4096);
    probe_align_seq_kernel<<<grid, kRedThreads, 0, s>>>(kl, logratio, gsq, window, rollout_len, B,
                                                        T, candidates, K, seq_stats, seq_full,
                                                        flags_out);
  }
  probe_align_batch_kernel<<<1, 96, 0, s>>>(seq_stats, seq_full, window, rollout_len, B, T,
                                            candidates, K, rho_star, batch_stats, L_next,
                                            flags_out);
  return cudaGetLastError();
}

}  // namespace adwin
