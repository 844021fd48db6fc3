// Device-side helpers shared by the kernels of the windowed OPD divergence library (sm_100a).
//
// Numerical scheme (all kernels): exponentials are taken in the base-2 domain against a running
// reference m2 that is an exact fp32 number >= every z*log2(e) seen so far,
//   e_k = 2^(fma(z_k, log2e, -m2)),
// so partial sums held by different threads / CTAs combine exactly through 2^(m2_i - M2).
// delta_k = (z_k - u_k) - dref is centred on the sampled token's log-odds so that the moments
// sum e*delta, sum e^2*delta^j stay well conditioned.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/adwin.h"

namespace adwin {

constexpr float kLog2e = 1.4426950408889634f;

// Bounds-checked build flavour (-DADWIN_CHECKED; compute-sanitizer's stand-in): every index the
// kernels form by hand -- shared-memory slots, ring cursors, exchange records, global pieces -- is
// tested before the access; a violation skips the access and raises ADWIN_DEV_BOUNDS in the status
// word.  Nothing traps.  In the ordinary build ADWIN_CHK(cond, status) is the constant `true` and
// the test disappears.  Usage:  if (ADWIN_CHK(i < n, p.status)) { ... a[i] ... }
#ifdef ADWIN_CHECKED
__device__ __forceinline__ bool chk_in_bounds(bool ok, int32_t* status) {
  if (!ok) atomicOr(status, (int32_t)ADWIN_DEV_BOUNDS);
  return ok;
}
#define ADWIN_CHK(cond, status) (::adwin::chk_in_bounds((cond), (status)))
#else
#define ADWIN_CHK(cond, status) (true)
#endif

// Everything the row kernels need; plain pointers, filled by the host entry point.
struct KlParams {
  const void* student;
  const void* teacher;
  int64_t B, T, V, ld;
  const int32_t* tokens;
  float alpha;
  int mode;   // adwin_grad_mode_t
  int flags;
  void* grad;          // may be null
  int64_t ld_grad;
  float* kl;
  float* logratio;
  float* gsq;          // may be null
  float* lse_s;        // may be null
  float* lse_t;        // may be null
  int32_t* status;
  // row map (workspace)
  const int32_t* range;    // [B] processed range P_b
  const int32_t* ewin;     // [B] effective window E_b
  const int64_t* offsets;  // [B+1] exclusive prefix sums of P_b
  // SAMPLED mode only: per-position coefficient that takes the place of c_t (the discounted
  // return-to-go of Eq. 3); null for the token-local estimator of Eq. 4
  const float* row_coef;
  // streaming kernel only: when set, positions t < skip_below[b] are left to another launch
  const int32_t* skip_below;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Element traits: N elements per 16-byte vector.
template <typename T>
struct Elem;
template <>
struct Elem<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void unpack(const uint4& v, float (&o)[4]) {
    o[0] = __uint_as_float(v.x);
    o[1] = __uint_as_float(v.y);
    o[2] = __uint_as_float(v.z);
    o[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ float load1(const void* p, int64_t i) {
    return static_cast<const float*>(p)[i];
  }
  __device__ static __forceinline__ void store1(void* p, int64_t i, float v) {
    static_cast<float*>(p)[i] = v;
  }
};
template <>
struct Elem<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void unpack(const uint4& v, float (&o)[8]) {
    o[0] = bf16lo(v.x);
    o[1] = bf16hi(v.x);
    o[2] = bf16lo(v.y);
    o[3] = bf16hi(v.y);
    o[4] = bf16lo(v.z);
    o[5] = bf16hi(v.z);
    o[6] = bf16lo(v.w);
    o[7] = bf16hi(v.w);
  }
  __device__ static __forceinline__ float load1(const void* p, int64_t i) {
    return __bfloat162float(static_cast<const __nv_bfloat16*>(p)[i]);
  }
  __device__ static __forceinline__ void store1(void* p, int64_t i, float v) {
    static_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
  }
};

// Per-thread online accumulators of one row (or one slice of a row).
struct RowAcc {
  float m2s, S, A;     // student: reference, sum e, sum e*delta
  float B0, B1, B2;    // sum e^2, sum e^2*delta, sum e^2*delta^2 (single-sweep gradient norm)
  float m2t, St;       // teacher: reference, sum e
  __device__ __forceinline__ void reset() {
    m2s = -INFINITY;
    m2t = -INFINITY;
    S = A = B0 = B1 = B2 = St = 0.f;
  }
};

// Fold N consecutive vocabulary entries into the accumulators.
template <int N, bool EXPAND>
__device__ __forceinline__ void acc_piece(const float (&z)[N], const float (&u)[N], float dref,
                                          RowAcc& a) {
  float zm = z[0], um = u[0];
#pragma unroll
  for (int i = 1; i < N; ++i) {
    zm = fmaxf(zm, z[i]);
    um = fmaxf(um, u[i]);
  }
  const float zl = zm * kLog2e, ul = um * kLog2e;
  if (zl > a.m2s) {
    const float f = ex2f(a.m2s - zl);
    a.S *= f;
    a.A *= f;
    if (EXPAND) {
      const float f2 = f * f;
      a.B0 *= f2;
      a.B1 *= f2;
      a.B2 *= f2;
    }
    a.m2s = zl;
  }
  if (ul > a.m2t) {
    a.St *= ex2f(a.m2t - ul);
    a.m2t = ul;
  }
#pragma unroll
  for (int i = 0; i < N; ++i) {
    const float e = ex2f(fmaf(z[i], kLog2e, -a.m2s));
    const float d = (z[i] - u[i]) - dref;
    a.S += e;
    a.A = fmaf(e, d, a.A);
    if (EXPAND) {
      const float e2 = e * e;
      const float e2d = e2 * d;
      a.B0 += e2;
      a.B1 += e2d;
      a.B2 = fmaf(e2d, d, a.B2);
    }
    a.St += ex2f(fmaf(u[i], kLog2e, -a.m2t));
  }
}

// Row totals brought to a common reference, and the per-row scalars derived from them.
struct RowTotals {
  float M2s, M2t;
  float S, A, B0, B1, B2, St;
};

struct RowScalars {
  float kl, c, lse_s, lse_t, gsq_expanded;
  float c0;      // E_p[delta] (centred): A/S
  float coef;    // alpha / S      (FULL_KL)   or  -alpha*c / S   (SAMPLED)
  float gy;      // SAMPLED: gradient entry at the sampled token, alpha*c*(1-p_y)
  bool nonfinite;
};

// Finalise one row from its totals (fp32; cheap enough for every thread to evaluate).
// zy, uy: logits at the sampled token (ignored when !y_valid); dref as used in the sweep.
//   lse = (M2 + log2 S) ln 2;  Delta = lse_s - lse_t = ((M2s - M2t) + log2(S/St)) ln 2;
//   E_p[delta] = A/S + dref
//   KL = E_p[delta] - Delta;   c = (z_y - u_y) - Delta
// The expanded squared norm sum p^2 (delta - E_p delta)^2 = (B2 - 2 c0 B1 + c0^2 B0) / S^2 is only
// used for rows whose gradient is not written.
// w: SAMPLED mode only, null or the address of a caller-supplied coefficient that takes the place
// of c (Eq. 3); it is read only on that branch.
__device__ __forceinline__ RowScalars finish_row(const RowTotals& t, float zy, float uy,
                                                 bool y_valid, float dref, float alpha, int mode,
                                                 const float* w = nullptr) {
  constexpr float kLn2f = 0.69314718055994531f;
  RowScalars r;
  const float l2s = log2f(t.S), l2t = log2f(t.St);
  r.lse_s = (t.M2s + l2s) * kLn2f;
  r.lse_t = (t.M2t + l2t) * kLn2f;
  // log2 S - log2 St as one logarithm of the ratio: both sums can be large against a shared
  // reference, and their separate logarithms would each carry an absolute error of an ulp of ~20.
  const float delta = ((t.M2s - t.M2t) + log2f(t.S / t.St)) * kLn2f;
  const float inv_s = 1.f / t.S;
  r.c0 = t.A * inv_s;
  r.kl = (r.c0 + dref) - delta;
  r.c = y_valid ? (zy - uy) - delta : __int_as_float(0x7fc00000);
  if (mode == ADWIN_GRAD_FULL_KL) {
    const float q = fmaf(r.c0, fmaf(r.c0, t.B0, -2.f * t.B1), t.B2) * (inv_s * inv_s);
    r.gsq_expanded = alpha * alpha * fmaxf(q, 0.f);
    r.coef = alpha * inv_s;
    r.gy = 0.f;
  } else {
    const float py = y_valid ? ex2f(fmaf(zy, kLog2e, -t.M2s)) * inv_s : __int_as_float(0x7fc00000);
    const float rest = fmaxf(fmaf(t.B0, inv_s * inv_s, -py * py), 0.f);  // sum_{k != y} p_k^2
    const float ac = alpha * (w ? *w : r.c);
    r.gsq_expanded = ac * ac * fmaf(1.f - py, 1.f - py, rest);
    r.coef = -ac * inv_s;
    r.gy = ac * (1.f - py);
  }
  r.nonfinite = !(isfinite(r.lse_s) && isfinite(r.lse_t));
  return r;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace adwin
