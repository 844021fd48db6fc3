// Shape-agnostic row kernel: one CTA per processed row, two sweeps over global memory.
//
// Sweep 1 streams z and u once and accumulates the online log-sum-exp statistics, sum e*delta
// (reverse KL) and the moments of the single-sweep gradient norm.  Sweep 2 (only for rows whose
// gradient is written) re-reads the row and writes g.  Any V, any row stride, any element
// alignment; 16-byte vector loads when the layout allows.  This is the fallback for layouts the
// staged cluster kernel does not take, and the reference point it is measured against.
#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {

// 128-thread CTAs, one row each, eight pairs of 16-byte loads in flight per thread: small CTAs put
// many independent rows on an SM, so one row's reduction overlaps the others' streaming (measured on
// the read-only pass at V = 151 936: 256 threads x 1 load 74 %, 256 x 8 81 %, 512 x 8 79 %,
// 128 x 16 78 %, 128 x 8 90 % of the measured copy bandwidth).
constexpr int kGenericThreads = 128;
constexpr int kGenericWarps = kGenericThreads / 32;
constexpr int kGenericUnroll = 8;

struct BlockScratch {
  float wm[2][kGenericWarps];
  float ws[6][kGenericWarps];
  float wq[kGenericWarps];
  RowScalars rs;
  RowTotals tot;
};

// Combine the per-thread accumulators of a CTA; every thread returns the same totals.
__device__ __forceinline__ RowTotals block_combine(const RowAcc& a, BlockScratch& sm) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float wms = warp_max(a.m2s), wmt = warp_max(a.m2t);
  const float fs = (a.m2s == -INFINITY) ? 0.f : ex2f(a.m2s - wms);
  const float ft = (a.m2t == -INFINITY) ? 0.f : ex2f(a.m2t - wmt);
  const float fs2 = fs * fs;
  float v[6] = {a.S * fs, a.A * fs, a.B0 * fs2, a.B1 * fs2, a.B2 * fs2, a.St * ft};
#pragma unroll
  for (int i = 0; i < 6; ++i) v[i] = warp_sum(v[i]);
  if (lane == 0) {
    sm.wm[0][warp] = wms;
    sm.wm[1][warp] = wmt;
#pragma unroll
    for (int i = 0; i < 6; ++i) sm.ws[i][warp] = v[i];
  }
  __syncthreads();
  RowTotals t;
  t.M2s = -INFINITY;
  t.M2t = -INFINITY;
#pragma unroll
  for (int w = 0; w < kGenericWarps; ++w) {
    t.M2s = fmaxf(t.M2s, sm.wm[0][w]);
    t.M2t = fmaxf(t.M2t, sm.wm[1][w]);
  }
  float acc[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int w = 0; w < kGenericWarps; ++w) {
    const float gs = (sm.wm[0][w] == -INFINITY) ? 0.f : ex2f(sm.wm[0][w] - t.M2s);
    const float gt = (sm.wm[1][w] == -INFINITY) ? 0.f : ex2f(sm.wm[1][w] - t.M2t);
    const float gs2 = gs * gs;
    acc[0] += sm.ws[0][w] * gs;
    acc[1] += sm.ws[1][w] * gs;
    acc[2] += sm.ws[2][w] * gs2;
    acc[3] += sm.ws[3][w] * gs2;
    acc[4] += sm.ws[4][w] * gs2;
    acc[5] += sm.ws[5][w] * gt;
  }
  t.S = acc[0];
  t.A = acc[1];
  t.B0 = acc[2];
  t.B1 = acc[3];
  t.B2 = acc[4];
  t.St = acc[5];
  return t;
}

template <typename TIn, typename TOut, bool VEC>
__global__ void __launch_bounds__(kGenericThreads) kl_generic_kernel(KlParams p) {
  __shared__ BlockScratch sm;
  constexpr int N = VEC ? Elem<TIn>::N : 1;
  const int64_t rows = p.B * p.T;
  const int tid = threadIdx.x;

  for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
    const int64_t b = r / p.T;
    const int t = (int)(r - b * p.T);
    if (t >= p.range[b]) continue;  // past the window: the row is never touched
    if (p.skip_below && t < p.skip_below[b]) continue;
    const bool write_grad = (p.grad != nullptr) && (t < p.ewin[b]);

    const char* zrow = static_cast<const char*>(p.student) + (size_t)r * p.ld * sizeof(TIn);
    const char* urow = static_cast<const char*>(p.teacher) + (size_t)r * p.ld * sizeof(TIn);
    const int y = p.tokens[r];
    const bool y_valid = (y >= 0) && ((int64_t)y < p.V);
    const int64_t yi = y_valid ? y : 0;
    const float zy = Elem<TIn>::load1(zrow, yi), uy = Elem<TIn>::load1(urow, yi);
    const float dref = zy - uy;

    RowAcc a;
    a.reset();
    const int64_t pieces = (p.V + N - 1) / N;  // VEC requires V % N == 0
    if (VEC) {
      // kGenericUnroll pairs of 16-byte loads in flight per thread; a row that is read only once
      // (no gradient) is streamed past the caches, otherwise sweep 2 should find it in L2
      const uint4* zs = reinterpret_cast<const uint4*>(zrow);
      const uint4* us = reinterpret_cast<const uint4*>(urow);
      int64_t i = tid;
      for (; i + (kGenericUnroll - 1) * kGenericThreads < pieces;
           i += kGenericUnroll * kGenericThreads) {
        uint4 zv[kGenericUnroll], uv[kGenericUnroll];
        if (!ADWIN_CHK(i + (kGenericUnroll - 1) * kGenericThreads < pieces && (i + (kGenericUnroll - 1) * kGenericThreads + 1) * N <= p.ld, p.status)) break;
#pragma unroll
        for (int h = 0; h < kGenericUnroll; ++h) {
          zv[h] = write_grad ? __ldg(zs + i + h * kGenericThreads) : __ldcs(zs + i + h * kGenericThreads);
          uv[h] = write_grad ? __ldg(us + i + h * kGenericThreads) : __ldcs(us + i + h * kGenericThreads);
        }
#pragma unroll
        for (int h = 0; h < kGenericUnroll; ++h) {
          float z[N], u[N];
          Elem<TIn>::unpack(zv[h], reinterpret_cast<float(&)[Elem<TIn>::N]>(z));
          Elem<TIn>::unpack(uv[h], reinterpret_cast<float(&)[Elem<TIn>::N]>(u));
          acc_piece<N, true>(z, u, dref, a);
        }
      }
      for (; i < pieces; i += kGenericThreads) {
        float z[N], u[N];
        if (!ADWIN_CHK((i + 1) * N <= p.ld, p.status)) break;
        const uint4 zv = write_grad ? __ldg(zs + i) : __ldcs(zs + i);
        const uint4 uv = write_grad ? __ldg(us + i) : __ldcs(us + i);
        Elem<TIn>::unpack(zv, reinterpret_cast<float(&)[Elem<TIn>::N]>(z));
        Elem<TIn>::unpack(uv, reinterpret_cast<float(&)[Elem<TIn>::N]>(u));
        acc_piece<N, true>(z, u, dref, a);
      }
    } else {
      for (int64_t i = tid; i < pieces; i += kGenericThreads) {
        float z[N], u[N];
        if (!ADWIN_CHK(i < p.ld, p.status)) break;
        z[0] = Elem<TIn>::load1(zrow, i);
        u[0] = Elem<TIn>::load1(urow, i);
        acc_piece<N, true>(z, u, dref, a);
      }
    }
    const RowTotals tot = block_combine(a, sm);
    if (tid == 0)
      sm.rs = finish_row(tot, zy, uy, y_valid, dref, p.alpha, p.mode,
                         p.row_coef ? p.row_coef + r : nullptr);
    __syncthreads();
    const RowScalars rs = sm.rs;

    float q = 0.f;
    if (write_grad) {
      char* grow = static_cast<char*>(p.grad) + (size_t)r * p.ld_grad * sizeof(TOut);
      const bool full = (p.mode == ADWIN_GRAD_FULL_KL);
      for (int64_t i = tid; i < pieces; i += kGenericThreads) {
        float z[N], u[N], g[N];
        if (!ADWIN_CHK((i + 1) * N <= p.V && (i + 1) * N <= p.ld_grad && (i + 1) * N <= p.ld, p.status)) break;
        if (VEC) {
          const uint4 zv = __ldg(reinterpret_cast<const uint4*>(zrow) + i);
          const uint4 uv = __ldg(reinterpret_cast<const uint4*>(urow) + i);
          Elem<TIn>::unpack(zv, reinterpret_cast<float(&)[Elem<TIn>::N]>(z));
          Elem<TIn>::unpack(uv, reinterpret_cast<float(&)[Elem<TIn>::N]>(u));
        } else {
          z[0] = Elem<TIn>::load1(zrow, i);
          u[0] = Elem<TIn>::load1(urow, i);
        }
#pragma unroll
        for (int j = 0; j < N; ++j) {
          const float e = ex2f(fmaf(z[j], kLog2e, -tot.M2s));
          if (full) {
            g[j] = e * (rs.coef * (((z[j] - u[j]) - dref) - rs.c0));
          } else {
            g[j] = (y_valid && i * N + j == yi) ? rs.gy : e * rs.coef;
          }
          q = fmaf(g[j], g[j], q);
        }
        if (VEC) {
          if (sizeof(TOut) == 4) {
            float4* o = reinterpret_cast<float4*>(grow) + i * (N / 4);
#pragma unroll
            for (int j = 0; j < N / 4; ++j)
              o[j] = make_float4(g[4 * j], g[4 * j + 1], g[4 * j + 2], g[4 * j + 3]);
          } else {
            if (N == 8) {
              uint4 o;
              o.x = pack_bf16x2(g[0], g[1]);
              o.y = pack_bf16x2(g[2], g[3]);
              o.z = pack_bf16x2(g[4], g[5]);
              o.w = pack_bf16x2(g[6], g[7]);
              reinterpret_cast<uint4*>(grow)[i] = o;
            } else {  // fp32 logits, bf16 gradient: 4 entries = 8 bytes
              uint2 o;
              o.x = pack_bf16x2(g[0], g[1]);
              o.y = pack_bf16x2(g[2], g[3]);
              reinterpret_cast<uint2*>(grow)[i] = o;
            }
          }
        } else {
          Elem<TOut>::store1(grow, i, g[0]);
        }
      }
      // fixed-order CTA sum of the squared entries
      q = warp_sum(q);
      if ((tid & 31) == 0) sm.wq[tid >> 5] = q;
      __syncthreads();
      q = 0.f;
#pragma unroll
      for (int w = 0; w < kGenericWarps; ++w) q += sm.wq[w];
    }
    if (tid == 0 && ADWIN_CHK(r >= 0 && r < rows, p.status)) {
      p.kl[r] = rs.kl;
      p.logratio[r] = rs.c;
      if (p.gsq) p.gsq[r] = write_grad ? q : rs.gsq_expanded;
      if (p.lse_s) p.lse_s[r] = rs.lse_s;
      if (p.lse_t) p.lse_t[r] = rs.lse_t;
      int bits = 0;
      if (!y_valid) bits |= ADWIN_DEV_TOKEN_RANGE;
      if (rs.nonfinite) bits |= ADWIN_DEV_NONFINITE;
      if (bits) atomicOr(p.status, bits);
    }
    __syncthreads();  // scratch is reused by the next row
  }
}

template <typename TIn, typename TOut>
static cudaError_t launch_t(const KlParams& p, bool vec, int grid, cudaStream_t s) {
  if (vec)
    kl_generic_kernel<TIn, TOut, true><<<grid, kGenericThreads, 0, s>>>(p);
  else
    kl_generic_kernel<TIn, TOut, false><<<grid, kGenericThreads, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_kl_generic(const KlParams& p, int dtype, int grad_dtype, bool vec, int sm_count,
                              cudaStream_t s) {
  const int64_t rows = p.B * p.T;
  if (rows == 0) return cudaSuccess;
  const int64_t cap = (int64_t)sm_count * 64;
  const int grid = (int)(rows < cap ? rows : cap);
  if (dtype == ADWIN_F32) {
    return grad_dtype == ADWIN_F32 ? launch_t<float, float>(p, vec, grid, s)
                                   : launch_t<float, __nv_bfloat16>(p, vec, grid, s);
  }
  return grad_dtype == ADWIN_F32 ? launch_t<__nv_bfloat16, float>(p, vec, grid, s)
                                 : launch_t<__nv_bfloat16, __nv_bfloat16>(p, vec, grid, s);
}

}  // namespace adwin
