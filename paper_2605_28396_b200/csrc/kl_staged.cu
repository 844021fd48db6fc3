// Staged cluster kernel: each logit byte is read from HBM once and the two sweeps of the method
// run concurrently on different warps.
//
// A thread-block cluster of CL CTAs (one CTA per SM) owns one processed row at a time; CTA `rank`
// owns a contiguous slice of the vocabulary, cut into chunks.  A producer lane streams the
// chunks of consecutive rows into a FIFO ring of shared-memory slots with bulk asynchronous copies
// (cp.async.bulk, one mbarrier per slot).  The ring holds a whole row slice plus a few slots in
// flight, so a chunk stays on chip from its first use to its last:
//   * the SWEEP-1 warps (10 of the 15 consumer warps) read each chunk as it lands and accumulate
//     the log-sum-exp statistics of both rows and sum e*delta (for rows without a gradient also
//     the moments of its squared norm); after the last chunk of a row every warp writes its
//     partial record into the exchange buffer of every CTA of the cluster (remote shared-memory
//     stores + remote mbarrier arrive) and goes straight on to the next row;
//   * the SWEEP-2 warps (the other 5) wait for the cl*10 records of a row, sum them in a fixed
//     order -- all of them, in every CTA, obtain bit-identical totals -- derive the row's scalars
//     and write the gradient from the chunks that are still in the ring, with 16-byte coalesced
//     stores, one row behind sweep 1.
// Sweep 1 needs two exponentials per entry and sweep 2 one, so the 10:5 split keeps the special-
// function pipe evenly loaded, HBM reads (sweep 1 of row i+1) and writes (sweep 2 of row i) flow
// at the same time, and the latency of the cluster exchange is hidden behind the other sweep.  A
// slot returns to the producer once every consumer warp has copied its pieces into registers.
//
// Exponentials are taken against a reference that the whole row shares (the logit of the sampled
// token), so partial sums add without rescaling.  If the sums overflow that reference, the
// sweep-2 warps of the cluster re-read the row from global memory with a running maximum and
// exchange once more among themselves.
//
// Clusters are persistent and walk the compact list of in-window rows; rows past the window cost
// nothing.  An mbarrier parity wait is only sound within one phase of the barrier, so every
// consumer warp observes every fill of every slot.  Every wait is bounded by a wall-clock limit;
// on expiry the CTA raises ADWIN_DEV_TIMEOUT, stops waiting anywhere, drains its own copies, and
// still reaches the final cluster barrier so that no peer is left behind.
#include <mutex>
#include <vector>

#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {

constexpr int kThreads = 512;        // 16 warps: the block keeps 128 registers per thread
constexpr int kNC = 15;              // consumer warps; warp 15 hosts the producer lane
constexpr int kProducerWarp = kNC;
constexpr int kP1 = 3;               // pieces of a chunk per sweep-1 thread
constexpr int kP2 = 6;               // pieces of a chunk per sweep-2 thread (two rounds of kP2/2)
constexpr int kMaxSlots = 32;
constexpr int kMaxCL = 8;
constexpr int kMaxRec1 = kMaxCL * 10;   // sweep-1 exchange records per row (cl * ns1)
constexpr int kMaxRec2 = kMaxCL * 5;    // sweep-2 records: squared norms, fallback (cl * ns2)
constexpr int kCtrlBytes = 9216;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s
constexpr float kSumLimit = 1.2676506e30f;        // 2^100: beyond it the shared reference is unsafe

struct StagedPlan {
  int cl;                 // cluster size
  int ns1, ns2;           // sweep-1 warps [0,ns1) and sweep-2 warps [ns1, ns1+ns2), ns1+ns2 == kNC
  int nch;                // chunks per slice (same for every rank)
  int nslot;              // ring slots, <= 2 * nch - 1; >= nch + 1 when a gradient is written
  int chunk_pieces;       // 16-byte pieces per chunk (per array)
  int per_rank_pieces;    // pieces per slice (last rank may own fewer)
  int num_clusters;
  uint32_t slot_bytes;    // 2 * chunk_pieces * 16
};

struct __align__(16) Ctrl {
  unsigned long long full[kMaxSlots];
  unsigned long long empty[kMaxSlots];
  unsigned long long xbar[2];    // sweep-1 records of a row are in (count cl*ns1)
  unsigned long long qbar[2];    // rank 0 only: squared-norm shares of a row are in (count cl*ns2)
  unsigned long long sbar;       // fallback records are in (count cl*ns2)
  int abort_flag;
  int pad;
  float xbuf[2][kMaxRec1][8];    // per row parity: one record per (rank, sweep-1 warp)
  float sbuf[2][kMaxRec2][8];    // records of the running-maximum fallback, by round parity
  float qbuf[2][kMaxRec2];       // rank 0 only
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
  __device__ __forceinline__ void reset() {
    S = A = St = B0 = B1 = B2 = 0ull;   // the bit pattern of {0.f, 0.f}
  }
};

// Sweep 1, rows whose gradient is written: e = 2^(z log2e - ref_s), delta = z - u uncentred.
template <int NP>
__device__ __forceinline__ void acc_grad(const f2_t (&Z)[NP], const f2_t (&U)[NP], f2_t nrefs,
                                         f2_t nreft, Acc2& a) {
  const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const f2_t E = ex2_2(fma2(Z[i], L2, nrefs));
    const f2_t D = fma2(U[i], NEG1, Z[i]);
    a.S = add2(a.S, E);
    a.A = fma2(E, D, a.A);
    a.St = add2(a.St, ex2_2(fma2(U[i], L2, nreft)));
  }
}

// Sweep 1, rows whose gradient is not written (probe rows): additionally the moments
// sum e^2 {1, delta, delta^2} of the single-sweep squared gradient norm, delta centred on dref.
template <int NP>
__device__ __forceinline__ void acc_probe(const f2_t (&Z)[NP], const f2_t (&U)[NP], f2_t nrefs,
                                          f2_t nreft, f2_t ndref, Acc2& a) {
  const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const f2_t E = ex2_2(fma2(Z[i], L2, nrefs));
    const f2_t D = add2(fma2(U[i], NEG1, Z[i]), ndref);
    a.S = add2(a.S, E);
    a.A = fma2(E, D, a.A);
    const f2_t E2 = mul2(E, E);
    const f2_t E2D = mul2(E2, D);
    a.B0 = add2(a.B0, E2);
    a.B1 = add2(a.B1, E2D);
    a.B2 = fma2(E2D, D, a.B2);
    a.St = add2(a.St, ex2_2(fma2(U[i], L2, nreft)));
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

template <typename TIn>
__device__ __forceinline__ void fetch_logits_at(const KlParams& p, int64_t r, int y, float& zy,
                                                float& uy) {
  const bool ok = (y >= 0) && ((int64_t)y < p.V);
  const int64_t yi = ok ? y : 0;
  zy = Elem<TIn>::load1(static_cast<const char*>(p.student) + (size_t)r * p.ld * sizeof(TIn), yi);
  uy = Elem<TIn>::load1(static_cast<const char*>(p.teacher) + (size_t)r * p.ld * sizeof(TIn), yi);
}

// Walks the compact list of processed rows.  The prefix sums of the current sequence are cached
// in registers, so locating a row touches global memory only when it crosses into a new sequence.
struct RowCursor {
  int64_t b, lo, hi;   // sequence, offsets[b], offsets[b+1]
  int32_t ew;          // effective window of sequence b
  __device__ __forceinline__ void init(const KlParams& p) {
    b = 0;
    lo = 0;
    hi = p.B > 0 ? p.offsets[1] : 0;
    ew = p.B > 0 ? p.ewin[0] : 0;
  }
  // Global row of processed-row ordinal n (ordinals must not decrease) and whether its gradient
  // is written.
  __device__ __forceinline__ int64_t locate(const KlParams& p, int64_t n, bool& wg) {
    while (n >= hi && b + 1 < p.B) {
      ++b;
      lo = hi;
      hi = p.offsets[b + 1];
      ew = p.ewin[b];
    }
    const int64_t t = n - lo;
    wg = (p.grad != nullptr) && (t < ew);
    return b * p.T + t;
  }
};

// Row metadata pipeline of one role: the current row (C) and the next one (N) in registers; the
// token of row i+2 and the logits at the token of row i+1 are requested while row i is processed.
template <typename TIn>
struct RowPipe {
  RowCursor cur;
  int64_t rC, rN;
  int yC, yN;
  float zyC, uyC;
  bool wgC, wgN;
  int64_t rNN;
  int yNN;
  float zyN, uyN;
  bool wgNN;
  int64_t base, step, count;
  __device__ __forceinline__ void fetch_row(const KlParams& p, int64_t i, int64_t& r, int& y,
                                            bool& wg) {
    if (i < count) {
      r = cur.locate(p, base + i * step, wg);
      y = p.tokens[r];
    }
  }
  __device__ __forceinline__ void init(const KlParams& p, int64_t base_, int64_t step_,
                                       int64_t count_) {
    base = base_;
    step = step_;
    count = count_;
    cur.init(p);
    rC = rN = 0;
    yC = yN = 0;
    zyC = uyC = 0.f;
    wgC = wgN = false;
    fetch_row(p, 0, rC, yC, wgC);
    if (count > 0) fetch_logits_at<TIn>(p, rC, yC, zyC, uyC);
    fetch_row(p, 1, rN, yN, wgN);
  }
  // At the top of iteration i: request what iterations i+1 and i+2 will need.
  __device__ __forceinline__ void prefetch(const KlParams& p, int64_t i) {
    zyN = uyN = 0.f;
    rNN = 0;
    yNN = 0;
    wgNN = false;
    if (i + 1 < count) fetch_logits_at<TIn>(p, rN, yN, zyN, uyN);
    fetch_row(p, i + 2, rNN, yNN, wgNN);
  }
  __device__ __forceinline__ void rotate() {
    rC = rN; yC = yN; wgC = wgN; zyC = zyN; uyC = uyN;
    rN = rNN; yN = yNN; wgN = wgNN;
  }
};

// Fixed-order sum over the lanes of a warp; every lane returns the same bits.
__device__ __forceinline__ float lane_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
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
  const int ns1 = plan.ns1, ns2 = plan.ns2;
  const int nch = plan.nch, nslot = plan.nslot;
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
    for (int s = 0; s < nslot; ++s) {
      mbar_init(smem_u32(&ctrl.full[s]), 1);
      mbar_init(smem_u32(&ctrl.empty[s]), kNC);
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(smem_u32(&ctrl.xbar[k]), cl * ns1);
      mbar_init(smem_u32(&ctrl.qbar[k]), cl * ns2);
    }
    mbar_init(smem_u32(&ctrl.sbar), cl * ns2);
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
  bool timed_out = false;

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer lane
    if (lane == 0) {
      int slot = 0;
      uint32_t phase = 0;
      int64_t fills = 0;
      RowCursor cur;
      cur.init(p);
      bool stop = false;
      for (int64_t i = 0; i < my_rows && !stop && !*abort; ++i) {
        bool wg_unused;
        const int64_t r = cur.locate(p, cluster_id + i * plan.num_clusters, wg_unused);
        const size_t row_off = ((size_t)r * p.ld + (size_t)piece0 * N) * sizeof(TIn);
        for (int j = 0; j < nch; ++j) {
          if (fills >= nslot &&
              !bounded_wait<false>(smem_u32(&ctrl.empty[slot]), phase ^ 1u, abort)) {
            stop = true;   // gave up: never overwrite a slot that may still be read
            break;
          }
          int np = pieces_in_chunk(j);
          np = np < 0 ? 0 : np;
          const uint32_t bytes = (uint32_t)np * 16u;
          const uint32_t bar = smem_u32(&ctrl.full[slot]);
          if (bytes == 0) {
            mbar_arrive(bar);
          } else {
            const size_t goff = row_off + (size_t)j * plan.chunk_pieces * 16;
            mbar_arrive_expect_tx(bar, 2u * bytes);
            const uint32_t dst = smem_u32(ring + (size_t)slot * plan.slot_bytes);
            bulk_load(dst, static_cast<const char*>(p.student) + goff, bytes, bar);
            bulk_load(dst + u_off, static_cast<const char*>(p.teacher) + goff, bytes, bar);
          }
          ++fills;
          if (++slot == nslot) {
            slot = 0;
            phase ^= 1u;
          }
        }
      }
      // Drain: every copy this CTA issued must have landed before its shared memory goes away.
      // Walk back over the last min(fills, nslot) fills.
      int64_t pending = fills < nslot ? fills : nslot;
      const uint64_t t0 = global_timer();
      bool gave_up = false;
      while (pending > 0) {
        if (--slot < 0) {
          slot = nslot - 1;
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
  } else if (warp < ns1) {
    // ------------------------------------------------------------------ sweep-1 warps
    const int t1 = ns1 * 32;                      // threads of this role
    const uint32_t toff = (uint32_t)tid * 16u;    // first of this thread's kP1 pieces in a chunk
    int slot = 0;
    uint32_t phase = 0;
    RowPipe<TIn> rp;
    rp.init(p, cluster_id, plan.num_clusters, my_rows);
    for (int64_t i = 0; i < my_rows; ++i) {
      rp.prefetch(p, i);
      const bool wg = rp.wgC;
      const float ref_s = rp.zyC * kLog2e, ref_t = rp.uyC * kLog2e;   // shared references
      const float dref = wg ? 0.f : rp.zyC - rp.uyC;                  // delta is centred on probe rows
      const f2_t nrefs = splat2(-ref_s), nreft = splat2(-ref_t), ndref = splat2(-dref);
      Acc2 a;
      a.reset();
      for (int j = 0; j < nch; ++j) {
        if (!bounded_wait<false>(smem_u32(&ctrl.full[slot]), phase, abort)) {
          timed_out = true;
          break;
        }
        // The thread's pieces go to registers and the warp is done with the slot at once.
        const char* sl = ring + (size_t)slot * plan.slot_bytes + toff;
        const int np = pieces_in_chunk(j);
        uint4 zr[kP1], ur[kP1];
#pragma unroll
        for (int h = 0; h < kP1; ++h) {
          if (tid + h * t1 < np) {
            zr[h] = *reinterpret_cast<const uint4*>(sl + (size_t)h * t1 * 16);
            ur[h] = *reinterpret_cast<const uint4*>(sl + u_off + (size_t)h * t1 * 16);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl.empty[slot]));
#pragma unroll
        for (int h = 0; h < kP1; ++h) {
          if (tid + h * t1 < np) {
            f2_t Z[NP], U[NP];
            Pairs<TIn>::make(zr[h], Z);
            Pairs<TIn>::make(ur[h], U);
            if (wg)
              acc_grad<NP>(Z, U, nrefs, nreft, a);
            else
              acc_probe<NP>(Z, U, nrefs, nreft, ndref, a);
          }
        }
        if (++slot == nslot) {
          slot = 0;
          phase ^= 1u;
        }
      }
      if (timed_out) break;
      // record = { S, A, St, B0, B1, B2, 0, 0 }: this warp's sums over its lanes, to every CTA
      const float v0 = lane_sum(hsum2(a.S)), v1 = lane_sum(hsum2(a.A)), v2 = lane_sum(hsum2(a.St));
      float v3 = 0.f, v4 = 0.f, v5 = 0.f;
      if (!wg) {
        v3 = lane_sum(hsum2(a.B0));
        v4 = lane_sum(hsum2(a.B1));
        v5 = lane_sum(hsum2(a.B2));
      }
      const int par = (int)(i & 1);
      if (lane < cl) {
        const uint32_t dst =
            map_to_rank(smem_u32(&ctrl.xbuf[par][rank * ns1 + warp][0]), (uint32_t)lane);
        remote_store4(dst, v0, v1, v2, v3);
        remote_store4(dst + 16, v4, v5, 0.f, 0.f);
        remote_arrive_release(map_to_rank(smem_u32(&ctrl.xbar[par]), (uint32_t)lane));
      }
      rp.rotate();
    }
  } else {
    // ------------------------------------------------------------------ sweep-2 warps
    const bool full_mode = (p.mode == ADWIN_GRAD_FULL_KL);
    const int w2 = warp - ns1;                    // warp index inside the role
    const int g2 = tid - ns1 * 32;                // thread index inside the role
    const int t2 = ns2 * 32;
    const int nrec1 = cl * ns1, nrec2 = cl * ns2;
    const uint32_t toff = (uint32_t)g2 * 16u;
    int slot = 0;
    uint32_t phase = 0;
    uint32_t safe_rounds = 0;   // completed fallback exchanges (parity of sbar)
    int64_t r_prev = 0;
    bool wg_prev = false;
    RowPipe<TIn> rp;
    rp.init(p, cluster_id, plan.num_clusters, my_rows);

    // rank 0, first sweep-2 warp: the squared norm of a written gradient row, once every
    // sweep-2 warp of the cluster has delivered its share
    auto collect_norm = [&](int64_t i_prev) -> bool {
      if (rank != 0 || w2 != 0) return true;
      const int par = (int)(i_prev & 1);
      if (!bounded_wait<true>(smem_u32(&ctrl.qbar[par]), (uint32_t)((i_prev >> 1) & 1), abort))
        return false;
      float s = 0.f;
      for (int rr = lane; rr < nrec2; rr += 32) s += ctrl.qbuf[par][rr];
      s = lane_sum(s);
      if (lane == 0 && wg_prev && p.gsq) p.gsq[r_prev] = s;
      return true;
    };

    for (int64_t i = 0; i < my_rows; ++i) {
      rp.prefetch(p, i);
      const bool wg = rp.wgC;
      const int64_t r = rp.rC;
      const int y = rp.yC;
      const float zy = rp.zyC, uy = rp.uyC;
      const bool y_valid = (y >= 0) && ((int64_t)y < p.V);
      const float ref_s = zy * kLog2e, ref_t = uy * kLog2e;
      const float dref = wg ? 0.f : zy - uy;
      const int par = (int)(i & 1);

      // Before this warp releases anything of row i: the two-deep norm buffer of row i-1 is read.
      if (i > 0 && !collect_norm(i - 1)) {
        timed_out = true;
        break;
      }
      if (!wg) {
        // Row without a gradient: sweep 2 has nothing to read, but every consumer warp observes
        // and releases every fill of a slot, and it does so as the chunks land, not after the
        // row's totals, so that such rows stream through a ring smaller than a row.
        for (int j = 0; j < nch; ++j) {
          if (!bounded_wait<false>(smem_u32(&ctrl.full[slot]), phase, abort)) {
            timed_out = true;
            break;
          }
          if (lane == 0) mbar_arrive(smem_u32(&ctrl.empty[slot]));
          if (++slot == nslot) {
            slot = 0;
            phase ^= 1u;
          }
        }
        if (timed_out) break;
      }

      // ---------------------------------------------------------------- totals of row i
      if (!bounded_wait<true>(smem_u32(&ctrl.xbar[par]), (uint32_t)((i >> 1) & 1), abort)) {
        timed_out = true;
        break;
      }
      RowTotals t;
      {
        float s[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int rr = lane; rr < nrec1; rr += 32) {
          const float4 x0 = *reinterpret_cast<const float4*>(&ctrl.xbuf[par][rr][0]);
          const float4 x1 = *reinterpret_cast<const float4*>(&ctrl.xbuf[par][rr][4]);
          s[0] += x0.x; s[1] += x0.y; s[2] += x0.z; s[3] += x0.w;
          s[4] += x1.x; s[5] += x1.y;
        }
        t.M2s = ref_s;
        t.M2t = ref_t;
        t.S = lane_sum(s[0]);
        t.A = lane_sum(s[1]);
        t.St = lane_sum(s[2]);
        t.B0 = t.B1 = t.B2 = 0.f;
        if (!wg) {
          t.B0 = lane_sum(s[3]);
          t.B1 = lane_sum(s[4]);
          t.B2 = lane_sum(s[5]);
        }
      }
      // ---------------------------------------------------------------- overflow fallback
      // The totals are identical in every sweep-2 warp of the cluster, so this branch is uniform.
      if (!(t.S < kSumLimit) || !(t.St < kSumLimit) || !(t.B0 < kSumLimit)) {
        // Few threads share a long slice here, so the running sums are kept in double and fed in
        // blocks of 8 pieces (each block accumulated in fp32 against its own running maximum).
        const char* zrow = static_cast<const char*>(p.student) + ((size_t)r * p.ld + (size_t)piece0 * N) * sizeof(TIn);
        const char* urow = static_cast<const char*>(p.teacher) + ((size_t)r * p.ld + (size_t)piece0 * N) * sizeof(TIn);
        double dS = 0.0, dA = 0.0, dB0 = 0.0, dB1 = 0.0, dB2 = 0.0, dSt = 0.0;
        float Ms = -INFINITY, Mt = -INFINITY;
        for (int64_t pc0 = g2; pc0 < my_pieces; pc0 += (int64_t)8 * t2) {
          RowAcc ra;
          ra.reset();
          for (int b8 = 0; b8 < 8; ++b8) {
            const int64_t pc = pc0 + (int64_t)b8 * t2;
            if (pc >= my_pieces) break;
            float z[N], u[N];
            const uint4 zv = __ldg(reinterpret_cast<const uint4*>(zrow) + pc);
            const uint4 uv = __ldg(reinterpret_cast<const uint4*>(urow) + pc);
            Elem<TIn>::unpack(zv, z);
            Elem<TIn>::unpack(uv, u);
            acc_piece<N, true>(z, u, dref, ra);
          }
          const float nMs = fmaxf(Ms, ra.m2s), nMt = fmaxf(Mt, ra.m2t);
          const double fo = (Ms == -INFINITY) ? 0.0 : exp2((double)(Ms - nMs));
          const double fn = (ra.m2s == -INFINITY) ? 0.0 : exp2((double)(ra.m2s - nMs));
          const double go = (Mt == -INFINITY) ? 0.0 : exp2((double)(Mt - nMt));
          const double gn = (ra.m2t == -INFINITY) ? 0.0 : exp2((double)(ra.m2t - nMt));
          dS = dS * fo + (double)ra.S * fn;
          dA = dA * fo + (double)ra.A * fn;
          dB0 = dB0 * (fo * fo) + (double)ra.B0 * (fn * fn);
          dB1 = dB1 * (fo * fo) + (double)ra.B1 * (fn * fn);
          dB2 = dB2 * (fo * fo) + (double)ra.B2 * (fn * fn);
          dSt = dSt * go + (double)ra.St * gn;
          Ms = nMs;
          Mt = nMt;
        }
        const float wms = warp_max(Ms), wmt = warp_max(Mt);
        const double fs = (Ms == -INFINITY) ? 0.0 : exp2((double)(Ms - wms));
        const double ft = (Mt == -INFINITY) ? 0.0 : exp2((double)(Mt - wmt));
        const float x1 = lane_sum((float)(dS * fs)), x2 = lane_sum((float)(dA * fs));
        const float x3 = lane_sum((float)(dB0 * fs * fs)), x4 = lane_sum((float)(dB1 * fs * fs));
        const float x5 = lane_sum((float)(dB2 * fs * fs)), x7 = lane_sum((float)(dSt * ft));
        if (lane < cl) {
          const uint32_t dst =
              map_to_rank(smem_u32(&ctrl.sbuf[safe_rounds & 1u][rank * ns2 + w2][0]), (uint32_t)lane);
          remote_store4(dst, wms, x1, x2, x3);
          remote_store4(dst + 16, x4, x5, wmt, x7);
          remote_arrive_release(map_to_rank(smem_u32(&ctrl.sbar), (uint32_t)lane));
        }
        if (!bounded_wait<true>(smem_u32(&ctrl.sbar), safe_rounds & 1u, abort)) {
          timed_out = true;
          break;
        }
        const float(*sb)[8] = ctrl.sbuf[safe_rounds & 1u];
        ++safe_rounds;
        float ms = -INFINITY, mt = -INFINITY;
        for (int rr = lane; rr < nrec2; rr += 32) {
          ms = fmaxf(ms, sb[rr][0]);
          mt = fmaxf(mt, sb[rr][6]);
        }
        t.M2s = warp_max(ms);
        t.M2t = warp_max(mt);
        float s[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int rr = lane; rr < nrec2; rr += 32) {
          const float* x = sb[rr];
          const float gs = (x[0] == -INFINITY) ? 0.f : ex2f(x[0] - t.M2s);
          const float gt = (x[6] == -INFINITY) ? 0.f : ex2f(x[6] - t.M2t);
          const float gs2 = gs * gs;
          s[0] += x[1] * gs; s[1] += x[2] * gs; s[2] += x[3] * gs2;
          s[3] += x[4] * gs2; s[4] += x[5] * gs2; s[5] += x[7] * gt;
        }
        t.S = lane_sum(s[0]);
        t.A = lane_sum(s[1]);
        t.B0 = lane_sum(s[2]);
        t.B1 = lane_sum(s[3]);
        t.B2 = lane_sum(s[4]);
        t.St = lane_sum(s[5]);
        // Round k+2 reuses the buffer of round k; it cannot start before round k+1 is complete,
        // which needs an arrival from every warp, made after it has read round k.
      }

      // ---------------------------------------------------------------- row scalars
      const RowScalars rs = finish_row(t, zy, uy, y_valid, dref, p.alpha, p.mode);
      if (w2 == 0 && lane == 0 && rank == 0) {
        p.kl[r] = rs.kl;
        p.logratio[r] = rs.c;
        if (p.gsq && !wg) p.gsq[r] = rs.gsq_expanded;
        if (p.lse_s) p.lse_s[r] = rs.lse_s;
        if (p.lse_t) p.lse_t[r] = rs.lse_t;
        int bits = 0;
        if (!y_valid) bits |= ADWIN_DEV_TOKEN_RANGE;
        if (rs.nonfinite) bits |= ADWIN_DEV_NONFINITE;
        if (bits) atomicOr(p.status, bits);
      }

      // ---------------------------------------------------------------- sweep 2
      float q = 0.f;
      if (wg) {
        const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
        const f2_t nM2s = splat2(-t.M2s), nc0 = splat2(-rs.c0), coef2 = splat2(rs.coef);
        const int64_t ypiece = y_valid ? ((int64_t)y / N - piece0) : -1;   // slice-relative
        char* gthread = static_cast<char*>(p.grad) +
                        ((size_t)r * p.ld_grad + (size_t)(piece0 + g2) * N) * sizeof(TOut);
        const size_t gstep = (size_t)plan.chunk_pieces * N * sizeof(TOut);
        f2_t Q = 0ull;
        for (int j = 0; j < nch; ++j) {
          if (!bounded_wait<false>(smem_u32(&ctrl.full[slot]), phase, abort)) {
            timed_out = true;
            break;
          }
          const char* sl = ring + (size_t)slot * plan.slot_bytes + toff;
          const int np = pieces_in_chunk(j);
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            constexpr int H = kP2 / 2;
            uint4 zr[H], ur[H];
#pragma unroll
            for (int h = 0; h < H; ++h) {
              const int hh = half * H + h;
              if (g2 + hh * t2 < np) {
                zr[h] = *reinterpret_cast<const uint4*>(sl + (size_t)hh * t2 * 16);
                ur[h] = *reinterpret_cast<const uint4*>(sl + u_off + (size_t)hh * t2 * 16);
              }
            }
            if (half == 1) {   // all pieces of the chunk are in registers: hand the slot back
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&ctrl.empty[slot]));
            }
#pragma unroll
            for (int h = 0; h < H; ++h) {
              const int hh = half * H + h;
              if (g2 + hh * t2 < np) {
                f2_t Z[NP], U[NP], G[NP];
                Pairs<TIn>::make(zr[h], Z);
                Pairs<TIn>::make(ur[h], U);
#pragma unroll
                for (int e = 0; e < NP; ++e) {
                  const f2_t E = ex2_2(fma2(Z[e], L2, nM2s));
                  if (full_mode) {
                    const f2_t D = add2(fma2(U[e], NEG1, Z[e]), nc0);
                    G[e] = mul2(E, mul2(D, coef2));
                  } else {
                    G[e] = mul2(E, coef2);
                  }
                }
                if (!full_mode && (int64_t)j * plan.chunk_pieces + g2 + hh * t2 == ypiece) {
                  const int e = (int)((int64_t)y - ((int64_t)y / N) * N);
#pragma unroll
                  for (int w = 0; w < NP; ++w) {
                    float lo, hi;
                    upk2(G[w], lo, hi);
                    if (e == 2 * w) lo = rs.gy;
                    if (e == 2 * w + 1) hi = rs.gy;
                    G[w] = pk2(lo, hi);
                  }
                }
#pragma unroll
                for (int e = 0; e < NP; ++e) Q = fma2(G[e], G[e], Q);
                store_pairs<TOut, NP>(gthread + (size_t)j * gstep + (size_t)hh * t2 * N * sizeof(TOut), G);
              }
            }
          }
          if (++slot == nslot) {
            slot = 0;
            phase ^= 1u;
          }
        }
        if (timed_out) break;
        q = lane_sum(hsum2(Q));
      }
      // this warp's share of the row's squared gradient norm, to rank 0
      if (lane == 0) {
        const uint32_t dst = map_to_rank(smem_u32(&ctrl.qbuf[par][rank * ns2 + w2]), 0u);
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst), "f"(q) : "memory");
        remote_arrive_release(map_to_rank(smem_u32(&ctrl.qbar[par]), 0u));
      }
      r_prev = r;
      wg_prev = wg;
      rp.rotate();
    }
    if (!timed_out && my_rows > 0 && !collect_norm(my_rows - 1)) timed_out = true;
  }
  if (timed_out && lane == 0) {
    atomicOr(p.status, ADWIN_DEV_TIMEOUT);
    // let the peers stop waiting as well
    for (int d = 0; d < cl; ++d)
      remote_store_u32(map_to_rank(smem_u32(&ctrl.abort_flag), (uint32_t)d), 1u);
  }
  // No CTA leaves while a peer may still write into its shared memory or arrive on its barriers.
  __syncwarp();
  cluster_sync_all();
}

// ---------------------------------------------------------------------------- host side
namespace {

constexpr int kSmemOptin = 232448;   // 227 KB: the per-CTA limit of sm_100

// Chunking for one cluster size; false when the ring cannot hold a slice plus two slots.
bool plan_for_cluster(int64_t pieces_total, int cl, bool has_grad, StagedPlan& plan) {
  const int64_t ring_bytes = kSmemOptin - kCtrlBytes;
  const int64_t per_rank = (pieces_total + cl - 1) / cl;
  if (per_rank * 16 > (int64_t)1 << 30) return false;
  // 10 warps take sweep 1 and 5 take sweep 2 (two exponentials per entry against one); a call
  // that writes no gradient has no sweep 2 and leaves one warp for the row scalars.
  const int ns1 = has_grad ? 10 : 14, ns2 = kNC - ns1;
  int64_t chunk_max = (int64_t)ns1 * 32 * kP1;
  if (has_grad && (int64_t)ns2 * 32 * kP2 < chunk_max) chunk_max = (int64_t)ns2 * 32 * kP2;
  int64_t nch = (per_rank + chunk_max - 1) / chunk_max;
  if (nch < 2 && per_rank >= 16) nch = 2;      // two chunks let consecutive rows overlap
  int64_t chunk_pieces = (per_rank + nch - 1) / nch;
  chunk_pieces = (chunk_pieces + 7) / 8 * 8;   // slots start on 128-byte boundaries
  if (chunk_pieces > chunk_max) chunk_pieces = chunk_max;
  nch = (per_rank + chunk_pieces - 1) / chunk_pieces;
  const int64_t slot_bytes = 2 * chunk_pieces * 16;
  int64_t nslot = ring_bytes / slot_bytes;
  if (nslot > kMaxSlots) nslot = kMaxSlots;
  // Sweep 1 may run ahead of sweep 2 by as many rows as the ring holds (two, when sweep 2 has
  // already released a row without a gradient); the exchange buffers and barriers are two deep,
  // so the ring must not hold two whole rows.
  if (nslot > 2 * nch - 1) nslot = 2 * nch - 1;
  if (nslot < 1) return false;
  if (has_grad && nslot < nch + (nch >= 2 ? 1 : 0)) return false;   // a row stays until sweep 2
  if ((int64_t)cl * ns1 > kMaxRec1 && has_grad) return false;
  if ((int64_t)cl * ns2 > kMaxRec2) return false;
  if (!has_grad && cl * ns1 > kMaxRec1) return false;
  plan.cl = cl;
  plan.ns1 = ns1;
  plan.ns2 = ns2;
  plan.nch = (int)nch;
  plan.nslot = (int)nslot;
  plan.chunk_pieces = (int)chunk_pieces;
  plan.per_rank_pieces = (int)per_rank;
  plan.slot_bytes = (uint32_t)slot_bytes;
  return true;
}

int plan_smem_bytes(const StagedPlan& plan) {
  return kCtrlBytes + plan.nslot * (int)plan.slot_bytes;
}

template <typename TIn, typename TOut>
cudaError_t max_clusters_for(const StagedPlan& plan, int sm_count, int& max_clusters) {
  auto kernel = kl_staged_kernel<TIn, TOut>;
  const int smem = plan_smem_bytes(plan);
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

// The cluster size is chosen once per (device, shape class): among the sizes whose slice fits the
// ring, the one that keeps the most SMs busy (cluster sizes that do not divide a GPC's SM count
// leave SMs idle), then the smaller cluster.
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
    const double score = (double)clusters * cl - 1e-3 * cl;
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
  const int smem = plan_smem_bytes(plan);
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
