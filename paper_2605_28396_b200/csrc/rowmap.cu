// Row map: effective windows, their prefix sums, and zero-fill of everything outside the
// processed range.
//
// E_b = min(W_b, R_b, T) is the effective prefix window of sequence b (the update is evaluated on
// the prefix of length L_t, and a rollout that ended early has fewer tokens).  P_b is the range the
// call processes: E_b, or R_b for a delayed full-rollout probe.  offsets[] = exclusive prefix sums
// of P_b gives the compact list of processed rows with no host round trip.
#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {

WorkspaceLayout workspace_layout(int64_t B) {
  auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
  WorkspaceLayout w;
  w.off_offsets = 256;
  w.off_range = up(w.off_offsets + (size_t)(B + 1) * sizeof(int64_t));
  w.off_ewin = up(w.off_range + (size_t)B * sizeof(int32_t));
  w.total = up(w.off_ewin + (size_t)B * sizeof(int32_t));
  w.off_offsets_win = w.total;
  w.total_ext = up(w.off_offsets_win + (size_t)(B + 1) * sizeof(int64_t));
  return w;
}

constexpr int kMapThreads = 1024;

__device__ __forceinline__ void clamp_lengths(int32_t w, int32_t r, int64_t T, int flags, int& E,
                                              int& P, bool& bad) {
  bad = (w < 0) || (r < 0) || ((int64_t)r > T);
  const int64_t rc = r < 0 ? 0 : ((int64_t)r > T ? T : r);
  const int64_t wc = w < 0 ? 0 : w;
  E = (int)(wc < rc ? wc : rc);
  P = (flags & ADWIN_RANGE_FULL) ? (int)rc : E;
}

// Block 0: scan.  Blocks >= 1: zero the per-token outputs of rows outside the processed range.
__global__ void __launch_bounds__(kMapThreads) rowmap_kernel(
    const int32_t* __restrict__ window, const int32_t* __restrict__ rollout_len, int64_t B,
    int64_t T, int flags, int64_t* offsets, int64_t* offsets_win, int32_t* range, int32_t* ewin,
    float* kl, float* logratio, float* gsq, float* lse_s, float* lse_t, int32_t* status) {
  if (blockIdx.x == 0) {
    __shared__ int64_t part[kMapThreads];
    const int tid = threadIdx.x;
    const int64_t per = (B + kMapThreads - 1) / kMapThreads;
    const int64_t b0 = tid * per, b1 = (b0 + per < B) ? b0 + per : B;
    int64_t sum = 0, sum_win = 0;
    bool any_bad = false;
    for (int64_t b = b0; b < b1; ++b) {
      int E, P;
      bool bad;
      clamp_lengths(window ? window[b] : (int32_t)T, rollout_len ? rollout_len[b] : (int32_t)T, T, flags, E, P, bad);
      any_bad |= bad;
      range[b] = P;
      ewin[b] = E;
      sum += P;
      sum_win += E;
    }
    part[tid] = sum;
    __syncthreads();
    // Hillis-Steele inclusive scan of the per-thread sums.
    for (int o = 1; o < kMapThreads; o <<= 1) {
      const int64_t v = (tid >= o) ? part[tid - o] : 0;
      __syncthreads();
      part[tid] += v;
      __syncthreads();
    }
    int64_t run = part[tid] - sum;
    for (int64_t b = b0; b < b1; ++b) {
      if (!ADWIN_CHK(b >= 0 && b < B && run >= 0 && run <= B * T, status)) break;
      offsets[b] = run;
      run += range[b];
    }
    if (tid == kMapThreads - 1) offsets[B] = part[tid];
    if (any_bad) atomicOr(status, ADWIN_DEV_WINDOW);
    if (offsets_win) {   // the same scan over the effective windows
      __syncthreads();
      part[tid] = sum_win;
      __syncthreads();
      for (int o = 1; o < kMapThreads; o <<= 1) {
        const int64_t v = (tid >= o) ? part[tid - o] : 0;
        __syncthreads();
        part[tid] += v;
        __syncthreads();
      }
      int64_t run_win = part[tid] - sum_win;
      for (int64_t b = b0; b < b1; ++b) {
        offsets_win[b] = run_win;
        run_win += ewin[b];
      }
      if (tid == kMapThreads - 1) offsets_win[B] = part[tid];
    }
    return;
  }
  const int64_t n = B * T;
  for (int64_t i = (int64_t)(blockIdx.x - 1) * kMapThreads + threadIdx.x; i < n;
       i += (int64_t)(gridDim.x - 1) * kMapThreads) {
    const int64_t b = i / T;
    const int t = (int)(i - b * T);
    int E, P;
    bool bad;
    clamp_lengths(window ? window[b] : (int32_t)T, rollout_len ? rollout_len[b] : (int32_t)T, T, flags, E, P, bad);
    if (t >= P && ADWIN_CHK(b < B && t >= 0 && t < T, status)) {
      kl[i] = 0.f;
      logratio[i] = 0.f;
      if (gsq) gsq[i] = 0.f;
      if (lse_s) lse_s[i] = 0.f;
      if (lse_t) lse_t[i] = 0.f;
    }
  }
}

cudaError_t launch_rowmap(const int32_t* window, const int32_t* rollout_len, int64_t B, int64_t T,
                          int flags, void* workspace, bool with_window_offsets, float* kl,
                          float* logratio, float* gsq, float* lse_s, float* lse_t, int32_t* status,
                          cudaStream_t s) {
  const WorkspaceLayout w = workspace_layout(B);
  char* base = static_cast<char*>(workspace);
  const int64_t n = B * T;
  int64_t fill_blocks = (n + kMapThreads - 1) / kMapThreads;
  if (fill_blocks > 1024) fill_blocks = 1024;
  if (fill_blocks < 1) fill_blocks = 1;
  rowmap_kernel<<<(int)(1 + fill_blocks), kMapThreads, 0, s>>>(
      window, rollout_len, B, T, flags, reinterpret_cast<int64_t*>(base + w.off_offsets),
      with_window_offsets ? reinterpret_cast<int64_t*>(base + w.off_offsets_win) : nullptr,
      reinterpret_cast<int32_t*>(base + w.off_range), reinterpret_cast<int32_t*>(base + w.off_ewin),
      kl, logratio, gsq, lse_s, lse_t, status);
  return cudaGetLastError();
}

// ADWIN_ZERO_TAIL: zero-fill the gradient rows t >= E_b.
template <typename TOut>
__global__ void __launch_bounds__(256) zero_tail_kernel(KlParams p) {
  const int64_t rows = p.B * p.T;
  for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
    const int64_t b = r / p.T;
    const int t = (int)(r - b * p.T);
    if (t < p.ewin[b]) continue;
    TOut* g = static_cast<TOut*>(p.grad) + (size_t)r * p.ld_grad;
    const bool vec = ((reinterpret_cast<uintptr_t>(g) & 15) == 0);
    constexpr int N = 16 / sizeof(TOut);
    int64_t k = 0;
    if (vec) {
      const int64_t nv = p.V / N;
      for (int64_t i = threadIdx.x; i < nv; i += blockDim.x)
        reinterpret_cast<uint4*>(g)[i] = make_uint4(0u, 0u, 0u, 0u);
      k = nv * N;
    }
    for (int64_t i = k + threadIdx.x; i < p.V; i += blockDim.x) Elem<TOut>::store1(g, i, 0.f);
  }
}

cudaError_t launch_zero_tail(const KlParams& p, int grad_dtype, cudaStream_t s) {
  const int64_t rows = p.B * p.T;
  if (rows == 0 || p.grad == nullptr) return cudaSuccess;
  const int grid = (int)(rows < 148 * 16 ? rows : 148 * 16);
  if (grad_dtype == ADWIN_F32)
    zero_tail_kernel<float><<<grid, 256, 0, s>>>(p);
  else
    zero_tail_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace adwin
