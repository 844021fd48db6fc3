// Staged cluster kernel: each logit byte is read from HBM once.
//
// A thread-block cluster of CL CTAs owns one processed row at a time; CTA `rank` owns a contiguous
// slice of the vocabulary.  Three kinds of warps share a CTA:
//   * one producer warp streams the slice of z and of u into a shared-memory ring with bulk
//     asynchronous copies (cp.async.bulk, one mbarrier per ring slot);
//   * 16 consumer warps make sweep 1 over the chunks as they land (log-sum-exp statistics of both
//     rows, sum e*delta, and for rows without a gradient the moments of its squared norm) and
//     sweep 2, which re-reads the slice from shared memory -- not from HBM -- and writes the
//     gradient with 16-byte coalesced stores;
//   * one finisher warp combines the consumer warps' partial sums, exchanges the CTA's record
//     with the CL-1 peers through distributed shared memory (remote stores + remote mbarrier
//     arrive), derives the row's scalars and publishes them to the consumers.
// When the ring holds two row slices (plan.lag == 1) the consumers run sweep 2 one row behind
// sweep 1:  S1(i) -> S2(i-1) -> S1(i+1) -> ...  so the exchange of row i is hidden behind sweep 2
// of row i-1 and no consumer warp ever waits for a peer CTA in steady state.  Otherwise
// (plan.lag == 0) sweep 2 of a row follows its own sweep 1.  A slot goes back to the producer as
// soon as its last reader is done with it, so the next rows' chunks stream in underneath the
// current rows' arithmetic.  Clusters are persistent and walk the compact list of in-window rows;
// rows past the window cost nothing.
//
// Ring invariant: chunks are numbered q = 0,1,2,... in the order rows are processed; chunk q lives
// in slot q % nslot and is fill number q / nslot of that slot.  full[slot] completes once per fill
// (producer arrive + transaction bytes), empty[slot] once per drain (one arrive per consumer warp).
// Per-row hand-offs are double buffered by row parity: partready (consumers -> finisher, sweep-1
// partials), rowready (finisher -> consumers, row scalars), qready (consumers -> finisher, squared
// norm of the written gradient), xbar (peer finishers -> finisher, exchanged records).
//
// Every wait is bounded by a wall-clock limit; on expiry the CTA raises ADWIN_DEV_TIMEOUT, stops
// waiting anywhere, drains its own copies, and still reaches the final cluster barrier so that no
// peer is left behind.
#include <mutex>
#include <vector>

#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {

constexpr int kNT = 512;             // consumer threads
constexpr int kNW = kNT / 32;        // consumer warps
constexpr int kProducerWarp = kNW;
constexpr int kFinisherWarp = kNW + 1;
constexpr int kThreads = kNT + 64;   // + producer warp + finisher warp
constexpr int kMaxSlots = 32;
constexpr int kMaxCL = 8;
constexpr int kXF = 12;              // floats per exchange record
constexpr int kCtrlBytes = 4096;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s

struct StagedPlan {
  int cl;                 // cluster size
  int lag;                // 1: sweep 2 runs one row behind sweep 1 (two row slices resident)
  int nslot;              // ring slots
  int nch;                // chunks per slice (same for every rank)
  int chunk_pieces;       // 16-byte pieces per chunk (per array)
  int per_rank_pieces;    // pieces per slice (last rank may own fewer)
  int num_clusters;
  uint32_t slot_bytes;    // 2 * chunk_pieces * 16
};

struct __align__(16) Ctrl {
  unsigned long long full[kMaxSlots];
  unsigned long long empty[kMaxSlots];
  unsigned long long xbar[2];
  unsigned long long partready[2];
  unsigned long long qready[2];
  unsigned long long rowready[2];
  int abort_flag;
  int pad[3];
  float xbuf[2][kMaxCL][kXF];
  float wpart[2][kNW][8];
  float wq[2][kNW];
  float rowres[2][8];
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// ---------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void remote_store4(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b),
               "f"(c), "f"(d)
               : "memory");
}
__device__ __forceinline__ void remote_store_u32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void remote_arrive_release(uint32_t addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr)
               : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes,
                                          uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::
                   : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint64_t global_timer() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns immediately (false) once the CTA has given up.
template <bool CLUSTER>
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
  if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
  if (*abort) return false;
  const uint64_t t0 = global_timer();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
    if (global_timer() - t0 > kWaitLimitNs) {
      *abort = 1;
      return false;
    }
  }
}

// Locate processed-row ordinal n: advance the monotone sequence pointer, return the global row.
__device__ __forceinline__ int64_t locate_row(const KlParams& p, int64_t n, int64_t& b) {
  while (b + 1 < p.B && p.offsets[b + 1] <= n) ++b;
  return b * p.T + (n - p.offsets[b]);
}

template <typename TIn>
__device__ __forceinline__ void load_piece(const char* slot, uint32_t u_off, int piece,
                                           float (&z)[Elem<TIn>::N], float (&u)[Elem<TIn>::N]) {
  const uint4 zv = *reinterpret_cast<const uint4*>(slot + (size_t)piece * 16);
  const uint4 uv = *reinterpret_cast<const uint4*>(slot + u_off + (size_t)piece * 16);
  Elem<TIn>::unpack(zv, z);
  Elem<TIn>::unpack(uv, u);
}

// ---------------------------------------------------------------------------- packed fp32 pairs
// sm_100 issues add/mul/fma on two fp32 lanes held in a 64-bit register pair in one slot
// (add.f32x2 / mul.f32x2 / fma.f32x2).  The sweeps are issue- and MUFU-bound, so all element-wise
// arithmetic is done on pairs; only ex2 (MUFU) is per lane.
typedef unsigned long long f2_t;

__device__ __forceinline__ f2_t pk2(float lo, float hi) {
  f2_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void upk2(f2_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f2_t fma2(f2_t a, f2_t b, f2_t c) {
  f2_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f2_t add2(f2_t a, f2_t b) {
  f2_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f2_t mul2(f2_t a, f2_t b) {
  f2_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f2_t ex2_2(f2_t x) {
  float a, b;
  upk2(x, a, b);
  return pk2(ex2f(a), ex2f(b));
}
__device__ __forceinline__ float hsum2(f2_t v) {
  float a, b;
  upk2(v, a, b);
  return a + b;
}
__device__ __forceinline__ f2_t splat2(float v) { return pk2(v, v); }

// A 16-byte piece as NP pairs of consecutive vocabulary entries.
template <typename T>
struct Pairs;
template <>
struct Pairs<__nv_bfloat16> {
  static constexpr int NP = 4;
  __device__ static __forceinline__ void make(const uint4& v, f2_t (&o)[4]) {
    o[0] = pk2(bf16lo(v.x), bf16hi(v.x));
    o[1] = pk2(bf16lo(v.y), bf16hi(v.y));
    o[2] = pk2(bf16lo(v.z), bf16hi(v.z));
    o[3] = pk2(bf16lo(v.w), bf16hi(v.w));
  }
};
template <>
struct Pairs<float> {
  static constexpr int NP = 2;
  __device__ static __forceinline__ void make(const uint4& v, f2_t (&o)[2]) {
    o[0] = pk2(__uint_as_float(v.x), __uint_as_float(v.y));
    o[1] = pk2(__uint_as_float(v.z), __uint_as_float(v.w));
  }
};

// Per-thread accumulators of one row slice, as pairs (even / odd entries).
struct Acc2 {
  f2_t S, A, St, B0, B1, B2;
  float m2s, m2t;
  __device__ __forceinline__ void reset() {
    S = A = St = B0 = B1 = B2 = 0ull;   // the bit pattern of {0.f, 0.f}
    m2s = -INFINITY;
    m2t = -INFINITY;
  }
};

template <int NP>
__device__ __forceinline__ void piece_max(const f2_t (&Z)[NP], const f2_t (&U)[NP], float& zm,
                                          float& um) {
  zm = -INFINITY;
  um = -INFINITY;
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    float a, b;
    upk2(Z[i], a, b);
    zm = fmaxf(zm, fmaxf(a, b));
    upk2(U[i], a, b);
    um = fmaxf(um, fmaxf(a, b));
  }
}

// Rows whose gradient is written: fixed references (set from the thread's first piece), no
// per-piece maximum, delta = z - u uncentred.  The caller checks the sums for overflow after the
// sweep and, if a later entry ran more than ~2^100 above the reference, redoes the slice with the
// online-maximum path (the slice is still resident in shared memory).
template <int NP>
__device__ __forceinline__ void acc_fast(const f2_t (&Z)[NP], const f2_t (&U)[NP], f2_t nm2s,
                                         f2_t nm2t, Acc2& a) {
  const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const f2_t E = ex2_2(fma2(Z[i], L2, nm2s));
    const f2_t D = fma2(U[i], NEG1, Z[i]);
    a.S = add2(a.S, E);
    a.A = fma2(E, D, a.A);
    a.St = add2(a.St, ex2_2(fma2(U[i], L2, nm2t)));
  }
}

// Rows whose gradient is not written (probe rows): online maximum per piece, plus the moments
// sum e^2 {1, delta, delta^2} of the single-sweep squared gradient norm, delta centred on dref.
template <int NP>
__device__ __forceinline__ void acc_probe(const f2_t (&Z)[NP], const f2_t (&U)[NP], float dref,
                                          Acc2& a) {
  float zm, um;
  piece_max<NP>(Z, U, zm, um);
  const float zl = zm * kLog2e, ul = um * kLog2e;
  if (zl > a.m2s) {
    const float f = ex2f(a.m2s - zl);
    const f2_t F = splat2(f), F2 = splat2(f * f);
    a.S = mul2(a.S, F);
    a.A = mul2(a.A, F);
    a.B0 = mul2(a.B0, F2);
    a.B1 = mul2(a.B1, F2);
    a.B2 = mul2(a.B2, F2);
    a.m2s = zl;
  }
  if (ul > a.m2t) {
    a.St = mul2(a.St, splat2(ex2f(a.m2t - ul)));
    a.m2t = ul;
  }
  const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
  const f2_t nm2s = splat2(-a.m2s), nm2t = splat2(-a.m2t), ndref = splat2(-dref);
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const f2_t E = ex2_2(fma2(Z[i], L2, nm2s));
    const f2_t D = add2(fma2(U[i], NEG1, Z[i]), ndref);
    a.S = add2(a.S, E);
    a.A = fma2(E, D, a.A);
    const f2_t E2 = mul2(E, E);
    const f2_t E2D = mul2(E2, D);
    a.B0 = add2(a.B0, E2);
    a.B1 = add2(a.B1, E2D);
    a.B2 = fma2(E2D, D, a.B2);
    a.St = add2(a.St, ex2_2(fma2(U[i], L2, nm2t)));
  }
}

template <typename TOut, int NP>
__device__ __forceinline__ void store_pairs(char* dst, const f2_t (&G)[NP]) {
  float g[2 * NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) upk2(G[i], g[2 * i], g[2 * i + 1]);
  if (sizeof(TOut) == 4) {
    float4* o = reinterpret_cast<float4*>(dst);
#pragma unroll
    for (int j = 0; j < NP / 2; ++j)
      __stcs(o + j, make_float4(g[4 * j], g[4 * j + 1], g[4 * j + 2], g[4 * j + 3]));
  } else if (NP == 4) {
    uint4 o;
    o.x = pack_bf16x2(g[0], g[1]);
    o.y = pack_bf16x2(g[2], g[3]);
    o.z = pack_bf16x2(g[4], g[5]);
    o.w = pack_bf16x2(g[6], g[7]);
    __stcs(reinterpret_cast<uint4*>(dst), o);
  } else {
    uint2 o;
    o.x = pack_bf16x2(g[0], g[1]);
    o.y = pack_bf16x2(g[2], g[3]);
    __stcs(reinterpret_cast<uint2*>(dst), o);
  }
}

// Row metadata shared by the consumer and finisher roles: which global row, whether its gradient
// is written, its sampled token and the two logits at that token.
struct RowCursor {
  int64_t b;   // monotone sequence pointer
  __device__ __forceinline__ void fetch_row(const KlParams& p, int64_t ordinal, bool in_range,
                                            int64_t& r, int& y, bool& wg) {
    if (in_range) {
      r = locate_row(p, ordinal, b);
      const int64_t bb = r / p.T;
      wg = (p.grad != nullptr) && ((r - bb * p.T) < p.ewin[bb]);
      y = p.tokens[r];
    }
  }
};

template <typename TIn>
__device__ __forceinline__ void fetch_logits_at(const KlParams& p, int64_t r, int y, float& zy,
                                                float& uy) {
  const bool ok = (y >= 0) && ((int64_t)y < p.V);
  const int64_t yi = ok ? y : 0;
  zy = Elem<TIn>::load1(static_cast<const char*>(p.student) + (size_t)r * p.ld * sizeof(TIn), yi);
  uy = Elem<TIn>::load1(static_cast<const char*>(p.teacher) + (size_t)r * p.ld * sizeof(TIn), yi);
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(kThreads, 1) kl_staged_kernel(KlParams p, StagedPlan plan) {
  constexpr int N = Elem<TIn>::N;
  constexpr int NP = Pairs<TIn>::NP;
  extern __shared__ __align__(128) char smem[];
  Ctrl& ctrl = *reinterpret_cast<Ctrl*>(smem);
  char* ring = smem + kCtrlBytes;
  volatile int* abort = &ctrl.abort_flag;

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const int cl = plan.cl;
  const int lag = plan.lag;
  const int64_t cluster_id = blockIdx.x / cl;
  const uint32_t u_off = (uint32_t)plan.chunk_pieces * 16u;

  // slice of this CTA, in 16-byte pieces
  const int64_t pieces_total = p.V / N;
  const int64_t piece0 = (int64_t)rank * plan.per_rank_pieces;
  int64_t my_pieces = pieces_total - piece0;
  my_pieces = my_pieces < 0 ? 0 : (my_pieces > plan.per_rank_pieces ? plan.per_rank_pieces : my_pieces);

  const int64_t total_rows = p.offsets[p.B];
  const int64_t my_rows =
      cluster_id < total_rows ? (total_rows - cluster_id + plan.num_clusters - 1) / plan.num_clusters : 0;

  if (tid == 0) {
    for (int s = 0; s < plan.nslot; ++s) {
      mbar_init(smem_u32(&ctrl.full[s]), 1);
      mbar_init(smem_u32(&ctrl.empty[s]), kNW);
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(smem_u32(&ctrl.xbar[k]), cl);
      mbar_init(smem_u32(&ctrl.partready[k]), kNW);
      mbar_init(smem_u32(&ctrl.qready[k]), kNW);
      mbar_init(smem_u32(&ctrl.rowready[k]), 1);
    }
    ctrl.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_sync_all();  // peers' barriers exist before any remote arrive

  // pieces of this CTA's slice that fall into chunk j (<= 0 for chunks past the slice end)
  auto pieces_in_chunk = [&](int j) -> int {
    const int left = (int)my_pieces - j * plan.chunk_pieces;
    return left < plan.chunk_pieces ? left : plan.chunk_pieces;
  };

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer warp
    if (lane == 0) {
      int slot = 0;
      uint32_t phase = 0;
      int64_t fills = 0;
      int64_t b = 0;
      for (int64_t i = 0; i < my_rows; ++i) {
        if (*abort) break;
        const int64_t r = locate_row(p, cluster_id + i * plan.num_clusters, b);
        const char* zrow = static_cast<const char*>(p.student) + ((size_t)r * p.ld + piece0 * N) * sizeof(TIn);
        const char* urow = static_cast<const char*>(p.teacher) + ((size_t)r * p.ld + piece0 * N) * sizeof(TIn);
        for (int j = 0; j < plan.nch; ++j) {
          if (fills >= plan.nslot) bounded_wait<false>(smem_u32(&ctrl.empty[slot]), phase ^ 1u, abort);
          int np = pieces_in_chunk(j);
          np = np < 0 ? 0 : np;
          const uint32_t bytes = (uint32_t)np * 16u;
          const uint32_t bar = smem_u32(&ctrl.full[slot]);
          if (bytes == 0) {
            mbar_arrive(bar);
          } else {
            mbar_arrive_expect_tx(bar, 2u * bytes);
            const uint32_t dst = smem_u32(ring + (size_t)slot * plan.slot_bytes);
            const size_t goff = (size_t)j * plan.chunk_pieces * 16;
            bulk_load(dst, zrow + goff, bytes, bar);
            bulk_load(dst + u_off, urow + goff, bytes, bar);
          }
          ++fills;
          if (++slot == plan.nslot) {
            slot = 0;
            phase ^= 1u;
          }
        }
      }
      // Drain: every copy this CTA issued must have landed before its shared memory goes away.
      // Walk back over the last min(fills, nslot) fills.
      int64_t pending = fills < plan.nslot ? fills : plan.nslot;
      const uint64_t t0 = global_timer();
      bool gave_up = false;
      while (pending > 0) {
        if (--slot < 0) {
          slot = plan.nslot - 1;
          phase ^= 1u;
        }
        const uint32_t bar = smem_u32(&ctrl.full[slot]);
        while (!gave_up && !mbar_try_wait(bar, phase)) {
          if (global_timer() - t0 > kWaitLimitNs) gave_up = true;
        }
        --pending;
      }
      if (gave_up) atomicOr(p.status, ADWIN_DEV_TIMEOUT);
    }
  } else if (warp == kFinisherWarp) {
    // ------------------------------------------------------------------ finisher warp
    // Iteration i < my_rows exchanges the sweep-1 record of row i; every iteration also carries the
    // CTA's share of the squared gradient norm of row i-1-lag (written by sweep 2), so 1+lag
    // trailing iterations deliver the last norms.  All CTAs of a cluster run the same iterations.
    RowCursor cur;
    cur.b = 0;
    int64_t rC = 0, rN = 0, rH1 = 0, rH2 = 0;
    int yC = 0, yN = 0;
    float zyC = 0.f, uyC = 0.f;
    bool wgC = false, wgN = false, wgH1 = false, wgH2 = false;
    cur.fetch_row(p, cluster_id, 0 < my_rows, rC, yC, wgC);
    if (my_rows > 0) fetch_logits_at<TIn>(p, rC, yC, zyC, uyC);
    cur.fetch_row(p, cluster_id + plan.num_clusters, 1 < my_rows, rN, yN, wgN);
    bool timed_out = false;
    const int64_t iters = my_rows > 0 ? my_rows + 1 + lag : 0;
    for (int64_t i = 0; i < iters; ++i) {
      const bool real = i < my_rows;
      // next rows' dependent loads, consumed one iteration later
      float zyN = 0.f, uyN = 0.f;
      int64_t rNN = 0;
      int yNN = 0;
      bool wgNN = false;
      if (i + 1 < my_rows) fetch_logits_at<TIn>(p, rN, yN, zyN, uyN);
      cur.fetch_row(p, cluster_id + (i + 2) * plan.num_clusters, i + 2 < my_rows, rNN, yNN, wgNN);

      const int par = (int)(i & 1);
      const uint32_t ph = (uint32_t)((i >> 1) & 1);
      float rec[8] = {-INFINITY, 0.f, 0.f, 0.f, 0.f, 0.f, -INFINITY, 0.f};
      if (real) {
        if (!bounded_wait<false>(smem_u32(&ctrl.partready[par]), ph, abort)) {
          timed_out = true;
          break;
        }
        // combine the consumer warps of this CTA (lane = source warp)
        const bool has = lane < kNW;
        const float* w = ctrl.wpart[par][has ? lane : 0];
        const float ms = has ? w[0] : -INFINITY, mt = has ? w[6] : -INFINITY;
        const float Ms = warp_max(ms), Mt = warp_max(mt);
        const float fs = (ms == -INFINITY) ? 0.f : ex2f(ms - Ms);
        const float ft = (mt == -INFINITY) ? 0.f : ex2f(mt - Mt);
        const float fs2 = fs * fs;
        rec[0] = Ms;
        rec[1] = warp_sum(has ? w[1] * fs : 0.f);
        rec[2] = warp_sum(has ? w[2] * fs : 0.f);
        rec[3] = warp_sum(has ? w[3] * fs2 : 0.f);
        rec[4] = warp_sum(has ? w[4] * fs2 : 0.f);
        rec[5] = warp_sum(has ? w[5] * fs2 : 0.f);
        rec[6] = Mt;
        rec[7] = warp_sum(has ? w[7] * ft : 0.f);
      }
      const int64_t jq = i - 1 - lag;               // row whose written-gradient norm is carried
      const int64_t rq = lag ? rH2 : rH1;
      const bool wgq = lag ? wgH2 : wgH1;
      float qcta = 0.f;
      if (jq >= 0) {
        if (!bounded_wait<false>(smem_u32(&ctrl.qready[jq & 1]), (uint32_t)((jq >> 1) & 1), abort)) {
          timed_out = true;
          break;
        }
        qcta = warp_sum(lane < kNW ? ctrl.wq[jq & 1][lane] : 0.f);
      }
      // exchange: lane d delivers this CTA's record to peer d, then arrives on d's barrier
      if (lane < cl) {
        const uint32_t dst = map_to_rank(smem_u32(&ctrl.xbuf[par][rank][0]), (uint32_t)lane);
        remote_store4(dst, rec[0], rec[1], rec[2], rec[3]);
        remote_store4(dst + 16, rec[4], rec[5], rec[6], rec[7]);
        remote_store4(dst + 32, qcta, 0.f, 0.f, 0.f);
        remote_arrive_release(map_to_rank(smem_u32(&ctrl.xbar[par]), (uint32_t)lane));
      }
      if (!bounded_wait<true>(smem_u32(&ctrl.xbar[par]), ph, abort)) {
        timed_out = true;
        break;
      }
      // combine the CL records (lane = source rank); identical in every CTA of the cluster
      RowTotals t;
      float qtot;
      {
        const bool has = lane < cl;
        const float* x = ctrl.xbuf[par][has ? lane : 0];
        const float ms = has ? x[0] : -INFINITY, mt = has ? x[6] : -INFINITY;
        t.M2s = warp_max(ms);
        t.M2t = warp_max(mt);
        const float fs = (ms == -INFINITY) ? 0.f : ex2f(ms - t.M2s);
        const float ft = (mt == -INFINITY) ? 0.f : ex2f(mt - t.M2t);
        const float fs2 = fs * fs;
        t.S = warp_sum(has ? x[1] * fs : 0.f);
        t.A = warp_sum(has ? x[2] * fs : 0.f);
        t.B0 = warp_sum(has ? x[3] * fs2 : 0.f);
        t.B1 = warp_sum(has ? x[4] * fs2 : 0.f);
        t.B2 = warp_sum(has ? x[5] * fs2 : 0.f);
        t.St = warp_sum(has ? x[7] * ft : 0.f);
        qtot = warp_sum(has ? x[8] : 0.f);
      }
      if (lane == 0) {
        if (rank == 0 && jq >= 0 && wgq && p.gsq) p.gsq[rq] = qtot;
        if (real) {
          const bool y_valid = (yC >= 0) && ((int64_t)yC < p.V);
          const float dref = wgC ? 0.f : zyC - uyC;   // sweep 1 centres delta only on probe rows
          const RowScalars rs = finish_row(t, zyC, uyC, y_valid, dref, p.alpha, p.mode);
          float* rr = ctrl.rowres[par];
          rr[0] = t.M2s;
          rr[1] = rs.c0;
          rr[2] = rs.coef;
          rr[3] = rs.gy;
          if (rank == 0) {
            p.kl[rC] = rs.kl;
            p.logratio[rC] = rs.c;
            if (p.gsq && !wgC) p.gsq[rC] = rs.gsq_expanded;
            if (p.lse_s) p.lse_s[rC] = rs.lse_s;
            if (p.lse_t) p.lse_t[rC] = rs.lse_t;
            int bits = 0;
            if (!y_valid) bits |= ADWIN_DEV_TOKEN_RANGE;
            if (rs.nonfinite) bits |= ADWIN_DEV_NONFINITE;
            if (bits) atomicOr(p.status, bits);
          }
          mbar_arrive(smem_u32(&ctrl.rowready[par]));   // release: the row scalars are visible
        }
      }
      __syncwarp();
      // rotate the metadata pipeline
      rH2 = rH1; wgH2 = wgH1;
      rH1 = rC; wgH1 = wgC;
      rC = rN; yC = yN; wgC = wgN; zyC = zyN; uyC = uyN;
      rN = rNN; yN = yNN; wgN = wgNN;
    }
    if (timed_out && lane == 0) {
      atomicOr(p.status, ADWIN_DEV_TIMEOUT);
      for (int d = 0; d < cl; ++d)
        remote_store_u32(map_to_rank(smem_u32(&ctrl.abort_flag), (uint32_t)d), 1u);
    }
  } else {
    // ------------------------------------------------------------------ consumer warps
    const bool full_mode = (p.mode == ADWIN_GRAD_FULL_KL);
    int s1_slot = 0, s2_slot = 0;
    uint32_t s1_phase = 0;
    bool timed_out = false;

    // metadata pipeline: row of this iteration's sweep 1 (C), the next one (N), the previous (P)
    RowCursor cur;
    cur.b = 0;
    int64_t rC = 0, rN = 0, rP = 0;
    int yC = 0, yN = 0, yP = 0;
    float zyC = 0.f, uyC = 0.f;
    bool wgC = false, wgN = false, wgP = false;
    cur.fetch_row(p, cluster_id, 0 < my_rows, rC, yC, wgC);
    if (my_rows > 0) fetch_logits_at<TIn>(p, rC, yC, zyC, uyC);
    cur.fetch_row(p, cluster_id + plan.num_clusters, 1 < my_rows, rN, yN, wgN);

    const uint32_t toff = (uint32_t)tid * 16u;   // this thread's piece inside every chunk
    const int64_t iters = my_rows > 0 ? my_rows + lag : 0;
    for (int64_t i = 0; i < iters; ++i) {
      float zyN = 0.f, uyN = 0.f;
      int64_t rNN = 0;
      int yNN = 0;
      bool wgNN = false;
      if (i + 1 < my_rows) fetch_logits_at<TIn>(p, rN, yN, zyN, uyN);
      cur.fetch_row(p, cluster_id + (i + 2) * plan.num_clusters, i + 2 < my_rows, rNN, yNN, wgNN);

      // ---------------------------------------------------------------- sweep 1 of row i
      if (i < my_rows) {
        Acc2 a;
        a.reset();
        const int slot0 = s1_slot;
        if (wgC) {
          // gradient row: fixed references from the first piece, checked once after the sweep
          f2_t nm2s = 0ull, nm2t = 0ull;
          bool have_ref = false;
          for (int j = 0; j < plan.nch; ++j) {
            if (!bounded_wait<false>(smem_u32(&ctrl.full[s1_slot]), s1_phase, abort)) timed_out = true;
            if (tid < pieces_in_chunk(j)) {
              const char* sl = ring + (size_t)s1_slot * plan.slot_bytes + toff;
              f2_t Z[NP], U[NP];
              Pairs<TIn>::make(*reinterpret_cast<const uint4*>(sl), Z);
              Pairs<TIn>::make(*reinterpret_cast<const uint4*>(sl + u_off), U);
              if (!have_ref) {
                float zm, um;
                piece_max<NP>(Z, U, zm, um);
                a.m2s = zm * kLog2e;
                a.m2t = um * kLog2e;
                nm2s = splat2(-a.m2s);
                nm2t = splat2(-a.m2t);
                have_ref = true;
              }
              acc_fast<NP>(Z, U, nm2s, nm2t, a);
            }
            if (++s1_slot == plan.nslot) {
              s1_slot = 0;
              s1_phase ^= 1u;
            }
          }
          // overflow / invalid reference: redo this thread's pieces with the online maximum
          constexpr float kSumLimit = 1.2676506e30f;   // 2^100
          if (!(hsum2(a.S) < kSumLimit) || !(hsum2(a.St) < kSumLimit)) {
            RowAcc ra;
            ra.reset();
            int s = slot0;
            for (int j = 0; j < plan.nch; ++j) {
              if (tid < pieces_in_chunk(j)) {
                float z[N], u[N];
                load_piece<TIn>(ring + (size_t)s * plan.slot_bytes, u_off, tid, z, u);
                acc_piece<N, false>(z, u, 0.f, ra);
              }
              if (++s == plan.nslot) s = 0;
            }
            a.reset();
            a.m2s = ra.m2s;
            a.m2t = ra.m2t;
            a.S = pk2(ra.S, 0.f);
            a.A = pk2(ra.A, 0.f);
            a.St = pk2(ra.St, 0.f);
          }
        } else {
          // probe row: nothing re-reads a chunk, so each slot goes back to the producer at once
          const float dref = zyC - uyC;
          for (int j = 0; j < plan.nch; ++j) {
            if (!bounded_wait<false>(smem_u32(&ctrl.full[s1_slot]), s1_phase, abort)) timed_out = true;
            if (tid < pieces_in_chunk(j)) {
              const char* sl = ring + (size_t)s1_slot * plan.slot_bytes + toff;
              f2_t Z[NP], U[NP];
              Pairs<TIn>::make(*reinterpret_cast<const uint4*>(sl), Z);
              Pairs<TIn>::make(*reinterpret_cast<const uint4*>(sl + u_off), U);
              acc_probe<NP>(Z, U, dref, a);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl.empty[s1_slot]));
            if (++s1_slot == plan.nslot) {
              s1_slot = 0;
              s1_phase ^= 1u;
            }
          }
        }
        if (timed_out) break;
        // warp partials -> finisher
        const float wms = warp_max(a.m2s), wmt = warp_max(a.m2t);
        const float fs = (a.m2s == -INFINITY) ? 0.f : ex2f(a.m2s - wms);
        const float ft = (a.m2t == -INFINITY) ? 0.f : ex2f(a.m2t - wmt);
        const float fs2 = fs * fs;
        const float v0 = warp_sum(hsum2(a.S) * fs), v1 = warp_sum(hsum2(a.A) * fs);
        const float v2 = warp_sum(hsum2(a.B0) * fs2), v3 = warp_sum(hsum2(a.B1) * fs2);
        const float v4 = warp_sum(hsum2(a.B2) * fs2), v5 = warp_sum(hsum2(a.St) * ft);
        if (lane == 0) {
          float* w = ctrl.wpart[i & 1][warp];
          w[0] = wms; w[1] = v0; w[2] = v1; w[3] = v2; w[4] = v3; w[5] = v4; w[6] = wmt; w[7] = v5;
          mbar_arrive(smem_u32(&ctrl.partready[i & 1]));
        }
      }

      // ---------------------------------------------------------------- sweep 2 of row i - lag
      const int64_t j2 = i - lag;
      if (j2 >= 0) {
        const int64_t r2 = lag ? rP : rC;
        const int y2 = lag ? yP : yC;
        const bool wg2 = lag ? wgP : wgC;
        const int par = (int)(j2 & 1);
        if (!bounded_wait<false>(smem_u32(&ctrl.rowready[par]), (uint32_t)((j2 >> 1) & 1), abort)) {
          timed_out = true;
          break;
        }
        float q = 0.f;
        if (wg2) {
          const float M2s = ctrl.rowres[par][0], c0 = ctrl.rowres[par][1], coef = ctrl.rowres[par][2],
                      gy = ctrl.rowres[par][3];
          const bool y_valid = (y2 >= 0) && ((int64_t)y2 < p.V);
          const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
          const f2_t nM2s = splat2(-M2s), nc0 = splat2(-c0), coef2 = splat2(coef);
          const int64_t ypiece = y_valid ? ((int64_t)y2 / N - piece0) : -1;   // slice-relative
          char* gthread = static_cast<char*>(p.grad) +
                          ((size_t)r2 * p.ld_grad + (size_t)(piece0 + tid) * N) * sizeof(TOut);
          const size_t gstep = (size_t)plan.chunk_pieces * N * sizeof(TOut);
          f2_t Q = 0ull;
          for (int j = 0; j < plan.nch; ++j) {
            if (tid < pieces_in_chunk(j)) {
              const char* sl = ring + (size_t)s2_slot * plan.slot_bytes + toff;
              f2_t Z[NP], U[NP], G[NP];
              Pairs<TIn>::make(*reinterpret_cast<const uint4*>(sl), Z);
              Pairs<TIn>::make(*reinterpret_cast<const uint4*>(sl + u_off), U);
#pragma unroll
              for (int k = 0; k < NP; ++k) {
                const f2_t E = ex2_2(fma2(Z[k], L2, nM2s));
                if (full_mode) {
                  const f2_t D = add2(fma2(U[k], NEG1, Z[k]), nc0);
                  G[k] = mul2(E, mul2(D, coef2));
                } else {
                  G[k] = mul2(E, coef2);
                }
              }
              if (!full_mode && (int64_t)j * plan.chunk_pieces + tid == ypiece) {
                const int e = (int)((int64_t)y2 - ((int64_t)y2 / N) * N);
#pragma unroll
                for (int k = 0; k < NP; ++k) {
                  float lo, hi;
                  upk2(G[k], lo, hi);
                  if (e == 2 * k) lo = gy;
                  if (e == 2 * k + 1) hi = gy;
                  G[k] = pk2(lo, hi);
                }
              }
#pragma unroll
              for (int k = 0; k < NP; ++k) Q = fma2(G[k], G[k], Q);
              store_pairs<TOut, NP>(gthread + (size_t)j * gstep, G);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl.empty[s2_slot]));
            if (++s2_slot == plan.nslot) s2_slot = 0;
          }
          q = warp_sum(hsum2(Q));
        } else {
          s2_slot = (s2_slot + plan.nch) % plan.nslot;   // released by sweep 1 already
        }
        if (lane == 0) {
          ctrl.wq[par][warp] = q;
          mbar_arrive(smem_u32(&ctrl.qready[par]));
        }
      }

      // rotate the metadata pipeline
      rP = rC; yP = yC; wgP = wgC;
      rC = rN; yC = yN; wgC = wgN; zyC = zyN; uyC = uyN;
      rN = rNN; yN = yNN; wgN = wgNN;
    }
    if (timed_out && lane == 0) {
      atomicOr(p.status, ADWIN_DEV_TIMEOUT);
      // let the peers stop waiting as well
      for (int d = 0; d < cl; ++d)
        remote_store_u32(map_to_rank(smem_u32(&ctrl.abort_flag), (uint32_t)d), 1u);
    }
  }
  // No CTA leaves while a peer may still write into its shared memory or arrive on its barriers.
  __syncwarp();
  cluster_sync_all();
}

// ---------------------------------------------------------------------------- host side
namespace {

constexpr int kSmemOptin = 232448;   // 227 KB: the per-CTA limit of sm_100

// Chunking of one cluster size; false when the slice does not fit the ring.
bool plan_for_cluster(int64_t pieces_total, int cl, bool has_grad, StagedPlan& plan) {
  const int64_t ring_bytes = kSmemOptin - kCtrlBytes;
  const int64_t per_rank = (pieces_total + cl - 1) / cl;
  if (per_rank * 16 > (int64_t)1 << 30) return false;
  int64_t nch, chunk_pieces;
  if (has_grad) {
    nch = (per_rank + kNT - 1) / kNT;
    chunk_pieces = (per_rank + nch - 1) / nch;
  } else {
    chunk_pieces = per_rank < kNT ? per_rank : kNT;
    nch = (per_rank + chunk_pieces - 1) / chunk_pieces;
  }
  chunk_pieces = (chunk_pieces + 7) / 8 * 8;   // slots start on 128-byte boundaries
  if (chunk_pieces > kNT) chunk_pieces = kNT;
  nch = (per_rank + chunk_pieces - 1) / chunk_pieces;
  const int64_t slot_bytes = 2 * chunk_pieces * 16;
  int64_t nslot = ring_bytes / slot_bytes;
  if (nslot > kMaxSlots) nslot = kMaxSlots;
  int lag = 0;
  if (has_grad) {
    if (2 * nch + 1 <= nslot) lag = 1;          // two row slices resident + one slot in flight
    else if (nch + 2 > nslot) return false;     // one row slice + two slots in flight
  } else {
    if (nslot < 2) return false;
    lag = 1;   // no slot is held for a second sweep: only the wait for the row scalars is deferred
  }
  plan.cl = cl;
  plan.lag = lag;
  plan.nslot = (int)nslot;
  plan.nch = (int)nch;
  plan.chunk_pieces = (int)chunk_pieces;
  plan.per_rank_pieces = (int)per_rank;
  plan.slot_bytes = (uint32_t)slot_bytes;
  return true;
}

template <typename TIn, typename TOut>
cudaError_t max_clusters_for(const StagedPlan& plan, int sm_count, int& max_clusters) {
  auto kernel = kl_staged_kernel<TIn, TOut>;
  const int smem = kCtrlBytes + plan.nslot * (int)plan.slot_bytes;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = plan.cl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3(plan.cl * sm_count);
  return cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg);
}

// The cluster size is chosen once per (device, shape class): among the sizes whose slice fits,
// prefer plans that hide the exchange (lag 1), then the one that keeps the most SMs busy (cluster
// sizes that do not divide a GPC's SM count leave SMs idle), then the smaller cluster.
struct PlanKey {
  int dev, dtype, grad_dtype, has_grad;
  int64_t pieces_total;
  bool operator==(const PlanKey& o) const {
    return dev == o.dev && dtype == o.dtype && grad_dtype == o.grad_dtype &&
           has_grad == o.has_grad && pieces_total == o.pieces_total;
  }
};
struct PlanEntry {
  PlanKey key;
  bool ok;
  StagedPlan plan;
};

template <typename TIn, typename TOut>
bool choose_plan(int64_t pieces_total, bool has_grad, int sm_count, StagedPlan& best) {
  double best_score = -1.0;
  for (int cl = 1; cl <= kMaxCL; ++cl) {
    StagedPlan plan = {};
    if (!plan_for_cluster(pieces_total, cl, has_grad, plan)) continue;
    int clusters = 0;
    if (max_clusters_for<TIn, TOut>(plan, sm_count, clusters) != cudaSuccess) {
      cudaGetLastError();
      continue;
    }
    if (clusters < 1) continue;
    const double ctas = (double)clusters * cl;
    const double score = ctas * ((plan.lag || !has_grad) ? 1.0 : 0.6) - 1e-3 * cl;
    if (score > best_score) {
      best_score = score;
      best = plan;
      best.num_clusters = clusters;
    }
  }
  return best_score > 0.0;
}

template <typename TIn, typename TOut>
cudaError_t launch_staged_t(const KlParams& p, int dtype, int grad_dtype, int sm_count,
                            cudaStream_t s) {
  static std::mutex mu;
  static std::vector<PlanEntry> cache;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const int N = dtype == ADWIN_F32 ? 4 : 8;
  const PlanKey key = {dev, dtype, grad_dtype, p.grad != nullptr ? 1 : 0, p.V / N};
  if (key.pieces_total < 1) return cudaErrorNotSupported;
  StagedPlan plan = {};
  bool ok = false, found = false;
  {
    std::lock_guard<std::mutex> lock(mu);
    for (const PlanEntry& c : cache)
      if (c.key == key) {
        plan = c.plan;
        ok = c.ok;
        found = true;
        break;
      }
    if (!found) {
      ok = choose_plan<TIn, TOut>(key.pieces_total, key.has_grad != 0, sm_count, plan);
      cache.push_back({key, ok, plan});
    }
  }
  if (!ok) return cudaErrorNotSupported;

  auto kernel = kl_staged_kernel<TIn, TOut>;
  const int smem = kCtrlBytes + plan.nslot * (int)plan.slot_bytes;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = plan.cl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int64_t rows = p.B * p.T;
  if (plan.num_clusters > rows) plan.num_clusters = (int)rows;
  cfg.gridDim = dim3(plan.cl * plan.num_clusters);
  return cudaLaunchKernelEx(&cfg, kernel, p, plan);
}

}  // namespace

cudaError_t launch_kl_staged(const KlParams& p, int dtype, int grad_dtype, int sm_count,
                             cudaStream_t s) {
  if (dtype == ADWIN_F32) {
    return grad_dtype == ADWIN_F32
               ? launch_staged_t<float, float>(p, dtype, grad_dtype, sm_count, s)
               : launch_staged_t<float, __nv_bfloat16>(p, dtype, grad_dtype, sm_count, s);
  }
  return grad_dtype == ADWIN_F32
             ? launch_staged_t<__nv_bfloat16, float>(p, dtype, grad_dtype, sm_count, s)
             : launch_staged_t<__nv_bfloat16, __nv_bfloat16>(p, dtype, grad_dtype, sm_count, s);
}

}  // namespace adwin
