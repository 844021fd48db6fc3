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

// 128-thread CTAs, one row each, five pairs of 16-byte loads in flight per thread: small CTAs put
// many independent rows on an SM, so one row's reduction overlaps the others' streaming (measured on
// the read-only pass at V = 151 936 with scalar arithmetic: 256 threads x 1 load 74 %, 256 x 8 81 %,
// 512 x 8 79 %, 128 x 16 78 %, 128 x 8 90 % of the measured copy bandwidth).  With sweep 1 on packed
// pairs the kernel wants more registers per thread; 5 loads at 5 CTAs per SM (<= 96 registers, no
// spills) measured best among 4..8 loads x 4..8 CTAs, 3 % faster than the scalar 128 x 8 form both
// on a cold GPU and in a back-to-back series (where every form runs ~12 % slower).
constexpr int kGenericThreads = 128;
constexpr int kGenericWarps = kGenericThreads / 32;
constexpr int kGenericUnroll = 5;
constexpr int kGenericMinBlocks = 5;   // CTAs per SM the register allocation leaves room for

struct BlockScratch {
  float wm[2][kGenericWarps];
  float ws[6][kGenericWarps];
  float wq[kGenericWarps];
  RowScalars rs;
  RowTotals tot;
};

// Sweep 1 on packed fp32 pairs: sm_100 issues add / mul / fma on two fp32 lanes of a 64-bit
// register pair in one slot, which halves the issue slots of the element-wise part (the sweep is
// bound by issue slots and the ex2 unit as much as by memory).  Even and odd entries of a piece
// accumulate separately; fold() adds the two lanes.
typedef unsigned long long pair_t;
__device__ __forceinline__ pair_t pair(float lo, float hi) {
  pair_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpair(pair_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ pair_t pfma(pair_t a, pair_t b, pair_t c) {
  pair_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ pair_t padd(pair_t a, pair_t b) {
  pair_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ pair_t pmul(pair_t a, pair_t b) {
  pair_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ pair_t pex2(pair_t x) {
  float a, b;
  unpair(x, a, b);
  return pair(ex2f(a), ex2f(b));
}
__device__ __forceinline__ float psum(pair_t v) {
  float a, b;
  unpair(v, a, b);
  return a + b;
}

struct PairAcc {
  float m2s, m2t;                  // running references, as in RowAcc
  pair_t S, A, B0, B1, B2, St;     // the sums of RowAcc, even / odd entries apart
  __device__ __forceinline__ void reset() {
    m2s = -INFINITY;
    m2t = -INFINITY;
    S = A = B0 = B1 = B2 = St = 0ull;   // the bit pattern of {0.f, 0.f}
  }
  __device__ __forceinline__ RowAcc fold() const {
    RowAcc a;
    a.m2s = m2s;
    a.m2t = m2t;
    a.S = psum(S);
    a.A = psum(A);
    a.B0 = psum(B0);
    a.B1 = psum(B1);
    a.B2 = psum(B2);
    a.St = psum(St);
    return a;
  }
};

// acc_piece<N, true> on pairs (N even).
template <int N>
__device__ __forceinline__ void acc_piece_pairs(const float (&z)[N], const float (&u)[N], float dref,
                                                PairAcc& a) {
  float zm = z[0], um = u[0];
#pragma unroll
  for (int i = 1; i < N; ++i) {
    zm = fmaxf(zm, z[i]);
    um = fmaxf(um, u[i]);
  }
  const float zl = zm * kLog2e, ul = um * kLog2e;
  if (zl > a.m2s) {
    const float f = ex2f(a.m2s - zl);
    const pair_t F = pair(f, f), F2 = pmul(F, F);
    a.S = pmul(a.S, F);
    a.A = pmul(a.A, F);
    a.B0 = pmul(a.B0, F2);
    a.B1 = pmul(a.B1, F2);
    a.B2 = pmul(a.B2, F2);
    a.m2s = zl;
  }
  if (ul > a.m2t) {
    const float f = ex2f(a.m2t - ul);
    a.St = pmul(a.St, pair(f, f));
    a.m2t = ul;
  }
  const pair_t L2 = pair(kLog2e, kLog2e), NEG1 = pair(-1.f, -1.f);
  const pair_t nms = pair(-a.m2s, -a.m2s), nmt = pair(-a.m2t, -a.m2t), ndref = pair(-dref, -dref);
#pragma unroll
  for (int i = 0; i < N; i += 2) {
    const pair_t Z = pair(z[i], z[i + 1]), U = pair(u[i], u[i + 1]);
    const pair_t E = pex2(pfma(Z, L2, nms));
    const pair_t D = padd(pfma(U, NEG1, Z), ndref);
    a.S = padd(a.S, E);
    a.A = pfma(E, D, a.A);
    const pair_t E2 = pmul(E, E);
    const pair_t E2D = pmul(E2, D);
    a.B0 = padd(a.B0, E2);
    a.B1 = padd(a.B1, E2D);
    a.B2 = pfma(E2D, D, a.B2);
    a.St = padd(a.St, pex2(pfma(U, L2, nmt)));
  }
}

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
__global__ void __launch_bounds__(kGenericThreads, kGenericMinBlocks) kl_generic_kernel(KlParams p) {
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
      PairAcc pa;
      pa.reset();
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
          acc_piece_pairs<N>(z, u, dref, pa);
        }
      }
      for (; i < pieces; i += kGenericThreads) {
        float z[N], u[N];
        if (!ADWIN_CHK((i + 1) * N <= p.ld, p.status)) break;
        const uint4 zv = write_grad ? __ldg(zs + i) : __ldcs(zs + i);
        const uint4 uv = write_grad ? __ldg(us + i) : __ldcs(us + i);
        Elem<TIn>::unpack(zv, reinterpret_cast<float(&)[Elem<TIn>::N]>(z));
        Elem<TIn>::unpack(uv, reinterpret_cast<float(&)[Elem<TIn>::N]>(u));
        acc_piece_pairs<N>(z, u, dref, pa);
      }
      a = pa.fold();
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
