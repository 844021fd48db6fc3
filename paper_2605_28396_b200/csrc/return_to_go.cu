// Discounted return-to-go of the per-token costs (Eq. 3 and the derivation in the appendix on the
// OPD gradient):  G_t = sum_{t' = t}^{E-1} gamma^(t'-t) c_t'  for t < E, 0 elsewhere, where E is the
// end of the sequence's processed range (the prefix window, or the rollout with ADWIN_RANGE_FULL).
// One block per sequence.  The recurrence G_t = c_t + gamma G_{t+1} is an affine map per position;
// every thread folds a contiguous segment from its end, thread 0 chains the 256 segment results
// from the last segment backwards, and every thread walks its segment again from the value at its
// end.  All sums are fp64 in a fixed order, so the result does not depend on the launch.
#include "adwin_internal.h"

namespace adwin {
namespace {

constexpr int kRtgThreads = 256;

__global__ void __launch_bounds__(kRtgThreads) return_to_go_kernel(
    const float* __restrict__ c, const int32_t* __restrict__ window,
    const int32_t* __restrict__ rollout_len, int64_t T, double gamma, int range_full,
    float* __restrict__ out) {
  __shared__ double seg_val[kRtgThreads];   // G at the segment start if G at its end were 0
  __shared__ double seg_mul[kRtgThreads];   // gamma^(segment length)
  __shared__ double seg_tail[kRtgThreads];  // G just past the segment's end
  const int64_t b = blockIdx.x;
  const int tid = threadIdx.x;
  int64_t R = rollout_len ? (int64_t)rollout_len[b] : T;
  R = R < 0 ? 0 : (R > T ? T : R);
  int64_t W = window[b];
  W = W < 0 ? 0 : W;
  const int64_t E = range_full ? R : (W < R ? W : R);
  const float* cb = c + b * T;
  float* ob = out + b * T;

  const int64_t len = (E + kRtgThreads - 1) / kRtgThreads;
  const int64_t t0 = (int64_t)tid * len;
  const int64_t t1 = t0 + len < E ? t0 + len : E;
  double acc = 0.0, mul = 1.0;
  for (int64_t t = t1 - 1; t >= t0; --t) {
    acc = (double)cb[t] + gamma * acc;
    mul *= gamma;
  }
  seg_val[tid] = acc;
  seg_mul[tid] = mul;
  __syncthreads();
  if (tid == 0) {
    double tail = 0.0;
    for (int i = kRtgThreads - 1; i >= 0; --i) {
      seg_tail[i] = tail;
      tail = seg_val[i] + seg_mul[i] * tail;
    }
  }
  __syncthreads();
  acc = seg_tail[tid];
  for (int64_t t = t1 - 1; t >= t0; --t) {
    acc = (double)cb[t] + gamma * acc;
    ob[t] = (float)acc;
  }
  for (int64_t t = E + tid; t < T; t += kRtgThreads) ob[t] = 0.f;
}

}  // namespace

cudaError_t launch_return_to_go(const float* logratio, const int32_t* window,
                                const int32_t* rollout_len, int64_t B, int64_t T, double gamma,
                                int flags, float* rtg, cudaStream_t s) {
  if (B <= 0 || T <= 0) return cudaSuccess;
  return_to_go_kernel<<<(unsigned)B, kRtgThreads, 0, s>>>(
      logratio, window, rollout_len, T, gamma, (flags & ADWIN_RANGE_FULL) ? 1 : 0, rtg);
  return cudaGetLastError();
}

}  // namespace adwin
