// Teacher-side drift diagnostics along student rollouts (Section 3.1).
//
// teacher_drift_kernel: for every position t < R_b one streaming sweep over the teacher row gives
//   H[b,t]    = entropy of softmax(u)            (the branching factor is BF = exp H)
//   rank[b,t] = 1 + #{k : u_k > u_y}             (rank of the sampled token under the teacher)
// The entropy is accumulated against a running maximum m as  H = log S + B/S  with
// S = sum e^(u-m) and B = sum e^(u-m) (m-u): both terms are non-negative, so nothing cancels.
// The row is read exactly once (2*V bytes of bf16), 16-byte loads, eight in flight per thread.
//
// worst_rank_kernel / drift_curves_kernel: the running worst rank of every rollout and, from it,
// the per-position survival fraction S_T^(k) and the mean branching factor.
#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {
namespace {

constexpr int kDriftThreads = 128;
constexpr int kDriftWarps = kDriftThreads / 32;
constexpr int kDriftUnroll = 8;
constexpr float kLn2 = 0.69314718055994531f;

struct DriftAcc {
  float m2;   // running maximum of u*log2(e)
  float S;    // sum 2^(u2 - m2)
  float Bq;   // sum 2^(u2 - m2) * (m2 - u2)      (in units of log2)
  int cnt;    // entries strictly above the sampled token's logit
  __device__ __forceinline__ void reset() {
    m2 = -INFINITY;
    S = 0.f;
    Bq = 0.f;
    cnt = 0;
  }
};

template <int N>
__device__ __forceinline__ void drift_piece(const float (&u)[N], float uy, DriftAcc& a) {
  float pm = u[0];
#pragma unroll
  for (int i = 1; i < N; ++i) pm = fmaxf(pm, u[i]);
  pm *= kLog2e;
  if (pm > a.m2) {   // move the reference: S' = f S,  B' = f (B + S (m' - m))
    const float f = (a.m2 == -INFINITY) ? 0.f : ex2f(a.m2 - pm);
    const float shift = (a.m2 == -INFINITY) ? 0.f : pm - a.m2;
    a.Bq = f * fmaf(a.S, shift, a.Bq);
    a.S *= f;
    a.m2 = pm;
  }
#pragma unroll
  for (int i = 0; i < N; ++i) {
    const float d = fmaf(-u[i], kLog2e, a.m2);   // m2 - u2 >= 0
    const float e = ex2f(-d);
    a.S += e;
    a.Bq = fmaf(e, d, a.Bq);
    a.cnt += (u[i] > uy) ? 1 : 0;
  }
}

struct DriftScratch {
  float m[kDriftWarps], s[kDriftWarps], b[kDriftWarps];
  int c[kDriftWarps];
};

template <typename TIn, bool VEC>
__global__ void __launch_bounds__(kDriftThreads) teacher_drift_kernel(
    const void* __restrict__ teacher, int64_t B, int64_t T, int64_t V, int64_t ld,
    const int32_t* __restrict__ tokens, const int32_t* __restrict__ rollout_len,
    float* __restrict__ entropy, int32_t* __restrict__ rank, int32_t* __restrict__ status) {
  __shared__ DriftScratch sm;
  constexpr int N = VEC ? Elem<TIn>::N : 1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t rows = B * T;
  for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
    const int64_t b = r / T;
    const int64_t t = r - b * T;
    int64_t R = rollout_len ? (int64_t)rollout_len[b] : T;
    if (R < 0 || R > T) {
      if (tid == 0 && t == 0) atomicOr(status, ADWIN_DEV_WINDOW);
      R = R < 0 ? 0 : T;
    }
    if (t >= R) {   // past the rollout: nothing is read
      if (tid == 0) {
        entropy[r] = 0.f;
        rank[r] = 0;
      }
      continue;
    }
    const char* urow = static_cast<const char*>(teacher) + (size_t)r * ld * sizeof(TIn);
    const int y = tokens[r];
    const bool y_valid = (y >= 0) && ((int64_t)y < V);
    const float uy = y_valid ? Elem<TIn>::load1(urow, y) : INFINITY;

    DriftAcc a;
    a.reset();
    const int64_t pieces = (V + N - 1) / N;   // VEC requires V % N == 0
    if (VEC) {
      const uint4* src = reinterpret_cast<const uint4*>(urow);
      int64_t i = tid;
      for (; i + (kDriftUnroll - 1) * kDriftThreads < pieces; i += kDriftUnroll * kDriftThreads) {
        uint4 v[kDriftUnroll];
        if (!ADWIN_CHK((i + (kDriftUnroll - 1) * kDriftThreads + 1) * N <= ld, status)) break;
#pragma unroll
        for (int k = 0; k < kDriftUnroll; ++k) v[k] = __ldcs(src + i + k * kDriftThreads);
#pragma unroll
        for (int k = 0; k < kDriftUnroll; ++k) {
          float u[Elem<TIn>::N];
          Elem<TIn>::unpack(v[k], u);
          drift_piece<Elem<TIn>::N>(u, uy, a);
        }
      }
      for (; i < pieces; i += kDriftThreads) {
        float u[Elem<TIn>::N];
        if (!ADWIN_CHK((i + 1) * N <= ld, status)) break;
        Elem<TIn>::unpack(__ldcs(src + i), u);
        drift_piece<Elem<TIn>::N>(u, uy, a);
      }
    } else {
      for (int64_t i = tid; i < pieces; i += kDriftThreads) {
        if (!ADWIN_CHK(i < ld, status)) break;
        float u[1] = {Elem<TIn>::load1(urow, i)};
        drift_piece<1>(u, uy, a);
      }
    }
    // warp, then block: bring the partial sums to the common maximum, fixed order
    const float wm = warp_max(a.m2);
    const float f = (a.m2 == -INFINITY) ? 0.f : ex2f(a.m2 - wm);
    const float sh = (a.m2 == -INFINITY) ? 0.f : wm - a.m2;
    float s = a.S * f, bq = f * fmaf(a.S, sh, a.Bq);
    int c = a.cnt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      s += __shfl_xor_sync(0xffffffffu, s, o);
      bq += __shfl_xor_sync(0xffffffffu, bq, o);
      c += __shfl_xor_sync(0xffffffffu, c, o);
    }
    if (lane == 0) {
      sm.m[warp] = wm;
      sm.s[warp] = s;
      sm.b[warp] = bq;
      sm.c[warp] = c;
    }
    __syncthreads();
    if (tid == 0) {
      float M = -INFINITY;
      for (int w = 0; w < kDriftWarps; ++w) M = fmaxf(M, sm.m[w]);
      float Ssum = 0.f, Bsum = 0.f;
      int C = 0;
      for (int w = 0; w < kDriftWarps; ++w) {
        const float g = (sm.m[w] == -INFINITY) ? 0.f : ex2f(sm.m[w] - M);
        const float d = (sm.m[w] == -INFINITY) ? 0.f : M - sm.m[w];
        Ssum += sm.s[w] * g;
        Bsum += g * fmaf(sm.s[w], d, sm.b[w]);
        C += sm.c[w];
      }
      const float H = (log2f(Ssum) + Bsum / Ssum) * kLn2;
      entropy[r] = H;
      rank[r] = y_valid ? C + 1 : 0;
      int bits = 0;
      if (!y_valid) bits |= ADWIN_DEV_TOKEN_RANGE;
      if (!isfinite(H)) bits |= ADWIN_DEV_NONFINITE;
      if (bits) atomicOr(status, bits);
    }
    __syncthreads();
  }
}

// Running worst rank of one rollout: worst[b,t] = max_{t' <= t} rank[b,t'] (ranks past the rollout
// are 0 and leave it unchanged).  One block per sequence; segment maxima, a serial pass over the
// segments (one per thread), then each segment again.
__global__ void __launch_bounds__(kDriftThreads) worst_rank_kernel(const int32_t* __restrict__ rank,
                                                                  int64_t T,
                                                                  int32_t* __restrict__ worst) {
  __shared__ int seg_max[kDriftThreads];
  __shared__ int seg_before[kDriftThreads];
  const int64_t b = blockIdx.x;
  const int tid = threadIdx.x;
  const int32_t* rb = rank + b * T;
  int32_t* wb = worst + b * T;
  const int64_t len = (T + kDriftThreads - 1) / kDriftThreads;
  const int64_t t0 = (int64_t)tid * len;
  const int64_t t1 = t0 + len < T ? t0 + len : T;
  int m = 0;
  for (int64_t t = t0; t < t1; ++t) m = max(m, rb[t]);
  seg_max[tid] = m;
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int i = 0; i < kDriftThreads; ++i) {
      seg_before[i] = run;
      run = max(run, seg_max[i]);
    }
  }
  __syncthreads();
  m = seg_before[tid];
  for (int64_t t = t0; t < t1; ++t) {
    m = max(m, rb[t]);
    wb[t] = m;
  }
}

// Per position: survival[j,t] = (1/B) #{b : worst[b,t] <= ks[j]},  n_active[t] = #{b : t < R_b},
// bf_mean[t] = mean over the active sequences of exp(entropy[b,t]) (0 when none is active).
// One thread per position, sequences in index order.
__global__ void __launch_bounds__(kDriftThreads) drift_curves_kernel(
    const float* __restrict__ entropy, const int32_t* __restrict__ worst,
    const int32_t* __restrict__ rollout_len, int64_t B, int64_t T, const int32_t* __restrict__ ks,
    int32_t K, double* __restrict__ survival, double* __restrict__ bf_mean,
    int32_t* __restrict__ n_active) {
  const int64_t t = (int64_t)blockIdx.x * kDriftThreads + threadIdx.x;
  if (t >= T) return;
  double bf = 0.0;
  int n = 0;
  for (int64_t b = 0; b < B; ++b) {
    int64_t R = rollout_len ? (int64_t)rollout_len[b] : T;
    R = R < 0 ? 0 : (R > T ? T : R);
    if (t < R) {
      bf += exp((double)entropy[b * T + t]);
      ++n;
    }
  }
  bf_mean[t] = n > 0 ? bf / (double)n : 0.0;
  n_active[t] = n;
  for (int j = 0; j < K; ++j) {
    const int k = ks[j];
    int alive = 0;
    for (int64_t b = 0; b < B; ++b) alive += (worst[b * T + t] <= k) ? 1 : 0;
    survival[(int64_t)j * T + t] = (double)alive / (double)B;
  }
}

}  // namespace

cudaError_t launch_teacher_drift(const void* teacher, int dtype, int64_t B, int64_t T, int64_t V,
                                 int64_t ld, const int32_t* tokens, const int32_t* rollout_len,
                                 float* entropy, int32_t* rank, int32_t* status, bool vec,
                                 int sm_count, cudaStream_t s) {
  const int64_t rows = B * T;
  if (rows <= 0) return cudaSuccess;
  // small CTAs, many more than are resident (rows are handed out in grid order): measured at
  // V = 151 936, 256 threads x 4 loads on 8 CTAs per SM reach 83 % of the copy bandwidth,
  // 128 x 8 on 16 per SM 89 %, 128 x 8 on 64 per SM 94 %
  int64_t grid = (int64_t)sm_count * 64;
  if (grid > rows) grid = rows;
#define ADWIN_DRIFT_LAUNCH(TIN, VEC)                                                      \
  teacher_drift_kernel<TIN, VEC><<<(unsigned)grid, kDriftThreads, 0, s>>>(                \
      teacher, B, T, V, ld, tokens, rollout_len, entropy, rank, status)
  if (dtype == ADWIN_F32) {
    if (vec) ADWIN_DRIFT_LAUNCH(float, true); else ADWIN_DRIFT_LAUNCH(float, false);
  } else {
    if (vec) ADWIN_DRIFT_LAUNCH(__nv_bfloat16, true); else ADWIN_DRIFT_LAUNCH(__nv_bfloat16, false);
  }
#undef ADWIN_DRIFT_LAUNCH
  return cudaGetLastError();
}

cudaError_t launch_drift_curves(const float* entropy, const int32_t* rank,
                                const int32_t* rollout_len, int64_t B, int64_t T,
                                const int32_t* ks, int32_t K, int32_t* worst, double* survival,
                                double* bf_mean, int32_t* n_active, cudaStream_t s) {
  if (T <= 0) return cudaSuccess;
  if (B > 0) worst_rank_kernel<<<(unsigned)B, kDriftThreads, 0, s>>>(rank, T, worst);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const unsigned blocks = (unsigned)((T + kDriftThreads - 1) / kDriftThreads);
  drift_curves_kernel<<<blocks, kDriftThreads, 0, s>>>(entropy, worst, rollout_len, B, T, ks, K,
                                                       survival, bf_mean, n_active);
  return cudaGetLastError();
}

}  // namespace adwin
