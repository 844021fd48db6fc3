// Staged cluster kernel: each logit byte is read from HBM once.
//
// A thread-block cluster of CL CTAs (one CTA per SM) owns one processed row at a time; CTA `rank`
// owns a contiguous slice of the vocabulary, cut into chunks of at most 1536 16-byte pieces per
// array.  Two sweeps are made over the slice: sweep 1 accumulates the log-sum-exp statistics of
// both rows and sum e*delta (plus, for rows without a gradient, the moments of its squared norm);
// sweep 2 writes the gradient with 16-byte coalesced stores.
//
// What bounds a streaming kernel is the number of bytes it keeps in flight (memory latency x
// bandwidth is about 60 KB per SM), so shared memory is split between two uses:
//   * `nres` chunks of the slice are RESIDENT: loaded once, read by sweep 1, kept, read again by
//     sweep 2 and only then handed back;
//   * the other chunks are STREAMED through a ring of `nring` slots that is always free to take
//     new loads: sweep 1 consumes and releases them, sweep 2 fetches them a second time -- a few
//     microseconds after the first read, so the second fetch is served by the L2 cache, not HBM.
// Resident and streamed chunks alternate along the slice, so HBM reads are in flight during both
// sweeps: the streamed part of row i during sweep 1 of row i, the resident part of row i+1 during
// sweep 2 of row i.  Two lanes of a producer warp issue the bulk asynchronous copies
// (cp.async.bulk, one mbarrier per slot): one feeds the ring, one refills the resident slots.
// A consumer warp copies its pieces of a chunk into registers and hands the slot back at once,
// so the refill is in flight while the arithmetic runs.
//
// 15 consumer warps do the arithmetic, each at its own pace: nothing but data dependences ties
// them together.  Exponentials are taken against a reference that the whole row shares (the
// logit of the sampled token), so partial sums add without rescaling.  After sweep 1 every warp
// writes its partial record into the exchange buffer of every CTA of the cluster (remote shared
// memory stores + remote mbarrier arrive), waits for the cl*15 records of the row, and sums them
// in a fixed order: all warps of all CTAs obtain bit-identical totals and derive the row's
// scalars themselves, with no hop through a leader.  Records also carry each warp's share of the
// squared norm of the gradient row written before.  If the sums overflow the shared reference (a
// sampled token more than ~69 nats below the row maximum), the cluster re-reads the row from
// global memory with a running maximum and exchanges once more.
//
// Clusters are persistent and walk the compact list of in-window rows; rows past the window cost
// nothing.  Every wait is bounded by a wall-clock limit; on expiry the CTA raises
// ADWIN_DEV_TIMEOUT, stops waiting anywhere, drains its own copies, and still reaches the final
// cluster barrier so that no peer is left behind.
#include <mutex>
#include <vector>

#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {

constexpr int kLeadMax = 2;          // chunks of the next row that sweep 1 takes during the exchange
constexpr int kNT = 480;             // consumer threads (512 in all: the block keeps 128 registers per thread)
constexpr int kNW = kNT / 32;        // consumer warps
constexpr int kG = 1;                // consumer groups: group g takes the chunks j with j % kG == g
constexpr int kP = 3;                // pieces of a chunk that each thread of the owning group handles
constexpr int kGT = kNT / kG;        // threads per group
constexpr int kGW = kNW / kG;        // warps per group = arrivals that release a resident slot
constexpr int kChunkMax = kGT * kP;  // 16-byte pieces per chunk (per array), at most
constexpr int kMaxChunks = 256;
constexpr int kProducerWarp = kNW;   // lane 0 feeds the stream ring, lane 1 refills the resident slots
constexpr int kThreads = kNT + 32;
constexpr int kMaxRes = 16;
constexpr int kMaxRing = 16;
constexpr int kMaxCL = 4;
constexpr int kMaxRec = kMaxCL * kNW;  // exchange records per row
constexpr int kCtrlBytes = 8192;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s
constexpr float kSumLimit = 1.2676506e30f;        // 2^100: beyond it the shared reference is unsafe

struct StagedPlan {
  int cl;                 // cluster size
  int nch;                // chunks per slice (same for every rank)
  int nres;               // resident chunks per slice
  int nring;              // stream-ring slots
  int lead;               // leading streamed chunks of a slice that sweep 1 takes one row ahead
  int chunk_pieces;       // 16-byte pieces per chunk (per array)
  int per_rank_pieces;    // pieces per slice (last rank may own fewer)
  int num_clusters;
  uint32_t slot_bytes;    // 2 * chunk_pieces * 16
  uint64_t wait_limit_ns; // limit of the handshake waits (the drain loops keep kWaitLimitNs)
  int tm;                 // 1: streamed chunks are kept in tensor memory between the sweeps
};

// What the consumers need to know about a row: which global row it is, whether its gradient is
// written, its sampled token and the two logits at that token (at element 0 when the token is out
// of range).  One lane loads these ahead of time so that the consumers hold no prefetch state.
constexpr int kMetaDepth = 4;
struct __align__(16) RowMeta {
  int64_t r;
  int y;
  int wg;
  float zy, uy;
  float w;      // caller-supplied row coefficient (0 when there is none)
  int pad;
};

struct __align__(16) Ctrl {
  unsigned long long res_full[kMaxRes];
  unsigned long long res_empty[kMaxRes];
  unsigned long long ring_full[kMaxRing];
  unsigned long long ring_empty[kMaxRing];
  unsigned long long xbar[2];
  unsigned long long sbar;
  int abort_flag;
  int pad;
  float xbuf[2][kMaxRec][8];   // per row parity: one record per (rank, warp)
  float sbuf[kMaxRec][8];      // records of the running-maximum fallback
  int16_t tab[kMaxChunks];     // chunk j -> resident slot k (>= 0) or -1 (streamed)
  int16_t ord[kMaxChunks];     // chunk j -> its ordinal among the streamed chunks
  uint32_t tmem_base;          // tensor-memory allocation (TM mode)
  RowMeta meta[kMetaDepth];    // row metadata, filled a few rows ahead by the metadata lane
  unsigned long long meta_full[kMetaDepth];
  unsigned long long meta_empty[kMetaDepth];
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
// Non-blocking test of a phase (try_wait may suspend the thread for a while before it answers).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
// L2 eviction priorities for the bulk copies: a chunk that will be fetched again by sweep 2 should
// outlive the chunks that are read only once.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load_hint(uint32_t dst, const void* src, uint32_t bytes,
                                               uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1], %2, [%3], %4;" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(pol)
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

// Tensor memory as a scratchpad (TM mode): 512 columns x 128 lanes x 32 bit = 256 KB per SM that a
// kernel without MMAs leaves idle.  A consumer thread parks the 16-byte pieces it has read in
// sweep 1 in its own lane (lane = 32*(warp%4) + laneid, the only lanes a warp may touch) and gets
// them back in sweep 2, so the streamed chunks are neither kept in shared memory nor fetched again.
constexpr int kTmCols = 512;
constexpr int kTmColsPerThread = 128;      // four consumer warps share the 512 columns of a lane group
__device__ __forceinline__ void tm_alloc(uint32_t dst_smem) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(kTmCols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tm_dealloc(uint32_t taddr) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(kTmCols) : "memory");
}
__device__ __forceinline__ void tm_store8(uint32_t taddr, const uint4& a, const uint4& b) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr),
               "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}
__device__ __forceinline__ void tm_load8(uint32_t taddr, uint4& a, uint4& b) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
               : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tm_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tm_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Bounded wait of one thread.  Returns immediately (false) once the CTA has given up.
template <bool CLUSTER>
__device__ __forceinline__ bool bounded_wait_lane(uint32_t bar, uint32_t parity,
                                                  volatile int* abort, uint64_t limit_ns) {
  if (limit_ns < 16) {   // diagnostic setting: a wait that is not satisfied right now runs out
    if (mbar_test_wait(bar, parity)) return true;
    *abort = 1;
    return false;
  }
  if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
  if (*abort) return false;
  const uint64_t t0 = global_timer();
  for (;;) {
    if (global_timer() - t0 > limit_ns) {
      *abort = 1;
      return false;
    }
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
  }
}
// The same for a whole (converged) consumer warp: every lane polls, and the warp takes ONE
// decision -- if any lane gave up, all do -- so that the warp-collective shuffles that follow a
// wait are never entered by a part of the warp only.
template <bool CLUSTER>
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, volatile int* abort,
                                             uint64_t limit_ns) {
  return __all_sync(0xffffffffu, bounded_wait_lane<CLUSTER>(bar, parity, abort, limit_ns)) != 0;
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
  __device__ __forceinline__ void fetch_row(const KlParams& p, int64_t ordinal, bool in_range,
                                            int64_t& r, int& y, bool& wg) {
    if (in_range) {
      r = locate(p, ordinal, wg);
      y = p.tokens[r];
    }
  }
};

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
__device__ __forceinline__ f2_t splat2(float v) { return pk2(v, v); }
__device__ __forceinline__ f2_t sub2(f2_t a, f2_t b) {
  f2_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x of a pair on the FMA pipe, to relieve the MUFU unit that bounds sweep 1.  x is clamped to
// [-120, 105] (below that the term is nil against a sum >= 1; at the upper end the result exceeds
// the limit that sends the row to the safe path), rounded to the nearest integer n by adding
// 1.5*2^23, 2^(x-n) comes from a degree-4 polynomial on [-1/2, 1/2] (relative error < 2.7e-6,
// mean 4e-8) and n is added to the exponent field.  A NaN comes out as a finite number: callers
// keep a second, unclamped use of the input so that it still poisons the row.
__device__ __forceinline__ f2_t ex2_poly2(f2_t x) {
  float a, b;
  upk2(x, a, b);
  a = fminf(fmaxf(a, -120.f), 105.f);
  b = fminf(fmaxf(b, -120.f), 105.f);
  const f2_t xc = pk2(a, b);
  const f2_t MG = splat2(12582912.f);
  const f2_t t = add2(xc, MG);
  const f2_t f = sub2(xc, sub2(t, MG));
  f2_t q = fma2(splat2(9.570101276e-03f), f, splat2(5.591785908e-02f));
  q = fma2(q, f, splat2(2.402474433e-01f));
  q = fma2(q, f, splat2(6.931217909e-01f));
  q = fma2(q, f, splat2(9.999992847e-01f));
  float tl, th, ql, qh;
  upk2(t, tl, th);
  upk2(q, ql, qh);
  const uint32_t rl = __float_as_uint(ql) + (__float_as_uint(tl) << 23);
  const uint32_t rh = __float_as_uint(qh) + (__float_as_uint(th) << 23);
  return pk2(__uint_as_float(rl), __uint_as_float(rh));
}
__device__ __forceinline__ float hsum2(f2_t v) {
  float a, b;
  upk2(v, a, b);
  return a + b;
}

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

// Teacher pairs per 16-byte piece whose exponential is evaluated on the FMA pipe: one of the four
// pairs of a bf16 piece (more than that and the FMA/ALU pipes become the limit, measured); none
// for fp32 logits, whose sweep has half the exponentials per byte and a 1e-5 tolerance.
template <typename T>
__host__ __device__ constexpr int kPolyPairs() { return sizeof(T) == 2 ? 1 : 0; }

// Sweep 1, rows whose gradient is written: e = 2^(z log2e - ref_s), delta = z - u uncentred.
// The first PT teacher pairs of a piece take their exponential from the polynomial (the teacher
// sum only enters through its logarithm, and delta still sees the unclamped logits).
template <int NP, int PT>
__device__ __forceinline__ void acc_grad(const f2_t (&Z)[NP], const f2_t (&U)[NP], f2_t nrefs,
                                         f2_t nreft, Acc2& a) {
  const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const f2_t E = ex2_2(fma2(Z[i], L2, nrefs));
    const f2_t D = fma2(U[i], NEG1, Z[i]);
    a.S = add2(a.S, E);
    a.A = fma2(E, D, a.A);
    const f2_t xt = fma2(U[i], L2, nreft);
    a.St = add2(a.St, (i < PT) ? ex2_poly2(xt) : ex2_2(xt));
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

// The two logits at the sampled token (at element 0 when the token is out of range).
template <typename TIn>
__device__ __forceinline__ void fetch_logits_at(const KlParams& p, int64_t r, int y, float& zy,
                                                float& uy) {
  const bool ok = (y >= 0) && ((int64_t)y < p.V);
  const int64_t yi = ok ? y : 0;
  zy = Elem<TIn>::load1(static_cast<const char*>(p.student) + (size_t)r * p.ld * sizeof(TIn), yi);
  uy = Elem<TIn>::load1(static_cast<const char*>(p.teacher) + (size_t)r * p.ld * sizeof(TIn), yi);
}

// Chunk j of a slice is resident iff the running count floor(j*nres/nch) steps at j: the nres
// resident chunks are spread evenly along the slice.  Returns the resident slot or -1.
__device__ __forceinline__ int resident_slot(int j, int nres, int nch) {
  const int a = (j * nres) / nch, b = ((j + 1) * nres) / nch;
  return b > a ? a : -1;
}

// Fixed-order sum over the lanes of a warp; every lane returns the same bits.
__device__ __forceinline__ float lane_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename TIn, typename TOut, bool TM>
__global__ void __launch_bounds__(kThreads, 1) kl_staged_kernel(KlParams p, StagedPlan plan) {
  constexpr int N = Elem<TIn>::N;
  constexpr int NP = Pairs<TIn>::NP;
  extern __shared__ __align__(128) char smem[];
  Ctrl& ctrl = *reinterpret_cast<Ctrl*>(smem);
  char* res_base = smem + kCtrlBytes;
  char* ring_base = res_base + (size_t)plan.nres * plan.slot_bytes;
  volatile int* abort = &ctrl.abort_flag;

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const int cl = plan.cl;
  const int nch = plan.nch, nres = plan.nres, nring = plan.nring;
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
    for (int s = 0; s < nres; ++s) {
      mbar_init(smem_u32(&ctrl.res_full[s]), 1);
      mbar_init(smem_u32(&ctrl.res_empty[s]), kGW);
    }
    for (int s = 0; s < nring; ++s) {
      mbar_init(smem_u32(&ctrl.ring_full[s]), 1);
      mbar_init(smem_u32(&ctrl.ring_empty[s]), kNW);
    }
    for (int j = 0, o = 0; j < nch; ++j) {
      ctrl.tab[j] = (int16_t)resident_slot(j, nres, nch);
      ctrl.ord[j] = (int16_t)o;
      if (ctrl.tab[j] < 0) ++o;
    }
    mbar_init(smem_u32(&ctrl.xbar[0]), cl * kNW);
    mbar_init(smem_u32(&ctrl.xbar[1]), cl * kNW);
    mbar_init(smem_u32(&ctrl.sbar), cl * kNW);
    for (int s = 0; s < kMetaDepth; ++s) {
      mbar_init(smem_u32(&ctrl.meta_full[s]), 1);
      mbar_init(smem_u32(&ctrl.meta_empty[s]), kNW);
    }
    ctrl.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (TM && warp == kProducerWarp) tm_alloc(smem_u32(&ctrl.tmem_base));   // the whole warp
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  cluster_sync_all();  // peers' barriers exist before any remote arrive

  // pieces of this CTA's slice that fall into chunk j (<= 0 for chunks past the slice end)
  auto pieces_in_chunk = [&](int j) -> int {
    const int left = (int)my_pieces - j * plan.chunk_pieces;
    return left < plan.chunk_pieces ? left : plan.chunk_pieces;
  };
  // issue the two bulk copies of chunk j of row r into a slot
  auto issue_chunk = [&](int64_t r, int j, char* slot, unsigned long long* full, uint64_t pol) {
    int np = pieces_in_chunk(j);
    np = np < 0 ? 0 : np;
    const uint32_t bytes = (uint32_t)np * 16u;
    const uint32_t bar = smem_u32(full);
    if (bytes == 0) {
      mbar_arrive(bar);
    } else {
      const size_t goff = ((size_t)r * p.ld + (size_t)piece0 * N) * sizeof(TIn) +
                          (size_t)j * plan.chunk_pieces * 16;
      // checked flavour: the copy lies inside the row's V elements and inside one slot
      if (!ADWIN_CHK(r >= 0 && r < p.B * p.T &&
                         ((size_t)piece0 * N) * sizeof(TIn) + (size_t)j * plan.chunk_pieces * 16 + bytes <=
                             (size_t)p.V * sizeof(TIn) &&
                         bytes <= u_off && 2u * u_off <= plan.slot_bytes &&
                         slot >= res_base &&
                         slot + plan.slot_bytes <= res_base + (size_t)(nres + nring) * plan.slot_bytes,
                     p.status)) {
        mbar_arrive(bar);   // keep the pipeline moving: the consumers see an empty fill
        return;
      }
      mbar_arrive_expect_tx(bar, 2u * bytes);
      const uint32_t dst = smem_u32(slot);
      bulk_load_hint(dst, static_cast<const char*>(p.student) + goff, bytes, bar, pol);
      bulk_load_hint(dst + u_off, static_cast<const char*>(p.teacher) + goff, bytes, bar, pol);
    }
  };

  if (warp == kProducerWarp && lane == 0) {
    // ------------------------------------------------------------------ ring producer
    if (nring > 0 && nres < nch) {
      int slot = 0;
      uint32_t phase = 0;
      int64_t fills = 0;
      RowCursor cur;
      cur.init(p);
      bool stop = false;
      // streamed chunks j in [j0, j1) of row r, in order
      const uint64_t pol_keep = l2_policy_evict_last();
      const uint64_t pol_once = l2_policy_evict_first();
      auto emit = [&](int64_t r, int j0, int j1, uint64_t pol) {
        for (int j = j0; j < j1 && !stop; ++j) {
          if (ctrl.tab[j] >= 0) continue;
          if (fills >= nring &&
              !bounded_wait_lane<false>(smem_u32(&ctrl.ring_empty[slot]), phase ^ 1u, abort, plan.wait_limit_ns)) {
            stop = true;   // gave up: never overwrite a slot that may still be read
            return;
          }
          issue_chunk(r, j, ring_base + (size_t)slot * plan.slot_bytes, &ctrl.ring_full[slot], pol);
          ++fills;
          if (++slot == nring) {
            slot = 0;
            phase ^= 1u;
          }
        }
      };
      // Order of the stream (the consumers walk it in the same order): sweep 1 of row i from
      // chunk `lead` on (row 0: from chunk 0), then the leading chunks of row i+1, then (rows
      // whose gradient is written) all streamed chunks of row i again for sweep 2.
      const int lead = plan.lead;
      for (int64_t i = 0; i < my_rows && !stop && !*abort; ++i) {
        bool wg, wg_next;
        const int64_t r = cur.locate(p, cluster_id + i * plan.num_clusters, wg);
        // first fetch of a chunk that sweep 2 fetches again: keep it in L2; last fetch: let it go
        emit(r, i == 0 ? 0 : lead, nch, (wg && !TM) ? pol_keep : pol_once);
        if (i + 1 < my_rows) {
          const int64_t rn = cur.locate(p, cluster_id + (i + 1) * plan.num_clusters, wg_next);
          emit(rn, 0, lead, wg_next ? pol_keep : pol_once);
        }
        if (wg && !TM) emit(r, 0, nch, pol_once);   // TM: sweep 2 reads tensor memory instead
      }
      // Drain: every copy this CTA issued must have landed before its shared memory goes away.
      int64_t pending = fills < nring ? fills : nring;
      const uint64_t t0 = global_timer();
      bool gave_up = false;
      while (pending > 0) {
        if (--slot < 0) {
          slot = nring - 1;
          phase ^= 1u;
        }
        const uint32_t bar = smem_u32(&ctrl.ring_full[slot]);
        while (!gave_up && !mbar_try_wait(bar, phase)) {
          if (global_timer() - t0 > kWaitLimitNs) gave_up = true;
        }
        --pending;
      }
      if (gave_up) atomicOr(p.status, ADWIN_DEV_TIMEOUT);
    }
  } else if (warp == kProducerWarp && lane == 1) {
    // ------------------------------------------------------------------ resident producer
    // Resident slot k takes resident chunk k of every row: fill number i belongs to row i and
    // waits for drain number i-1 (sweep 2 of row i-1, or its sweep 1 if no gradient is written).
    if (nres > 0) {
      RowCursor cur;
      cur.init(p);
      const uint64_t pol_once = l2_policy_evict_first();   // resident chunks are fetched once
      int64_t last_row = -1;   // last row some slot was filled for, and how many slots got it
      int last_k = 0;
      for (int64_t i = 0; i < my_rows && !*abort; ++i) {
        bool wg_unused;
        const int64_t r = cur.locate(p, cluster_id + i * plan.num_clusters, wg_unused);
        for (int j = 0; j < nch; ++j) {
          const int k = ctrl.tab[j];
          if (k < 0) continue;
          if (i > 0 &&
              !bounded_wait_lane<false>(smem_u32(&ctrl.res_empty[k]), (uint32_t)((i - 1) & 1), abort, plan.wait_limit_ns))
            break;   // gave up: never overwrite a slot that may still be read
          issue_chunk(r, j, res_base + (size_t)k * plan.slot_bytes, &ctrl.res_full[k], pol_once);
          last_row = i;
          last_k = k + 1;
        }
      }
      // Drain: the last fill of every resident slot must have landed before the CTA exits
      // (slots k < last_k were filled for last_row, the others for the row before).
      const uint64_t t0 = global_timer();
      bool gave_up = false;
      for (int k = 0; k < nres; ++k) {
        const int64_t fill = k < last_k ? last_row : last_row - 1;
        if (fill < 0) continue;
        const uint32_t bar = smem_u32(&ctrl.res_full[k]);
        while (!gave_up && !mbar_try_wait(bar, (uint32_t)(fill & 1))) {
          if (global_timer() - t0 > kWaitLimitNs) gave_up = true;
        }
      }
      if (gave_up) atomicOr(p.status, ADWIN_DEV_TIMEOUT);
    }
  } else if (warp == kProducerWarp && lane == 2) {
    // ------------------------------------------------------------------ metadata lane
    RowCursor cur;
    cur.init(p);
    for (int64_t i = 0; i < my_rows && !*abort; ++i) {
      const int ms = (int)(i % kMetaDepth);
      if (i >= kMetaDepth &&
          !bounded_wait_lane<false>(smem_u32(&ctrl.meta_empty[ms]),
                               (uint32_t)((i / kMetaDepth - 1) & 1), abort, plan.wait_limit_ns))
        break;
      bool wg;
      const int64_t r = cur.locate(p, cluster_id + i * plan.num_clusters, wg);
      const int y = p.tokens[r];
      float zy, uy;
      fetch_logits_at<TIn>(p, r, y, zy, uy);
      if (!ADWIN_CHK(ms >= 0 && ms < kMetaDepth && r >= 0 && r < p.B * p.T, p.status)) break;
      RowMeta& m = ctrl.meta[ms];
      m.r = r;
      m.y = y;
      m.wg = wg ? 1 : 0;
      m.zy = zy;
      m.uy = uy;
      m.w = p.row_coef ? p.row_coef[r] : 0.f;
      mbar_arrive(smem_u32(&ctrl.meta_full[ms]));   // release: the fields are visible
    }
  } else if (warp < kNW) {
    // ------------------------------------------------------------------ consumer warps
    const bool full_mode = (p.mode == ADWIN_GRAD_FULL_KL);
    const int nrec = cl * kNW;
    int rc_slot = 0;            // ring cursor
    uint32_t rc_phase = 0;
    uint32_t safe_rounds = 0;   // completed fallback exchanges (parity of sbar)
    bool timed_out = false;
    float q_prev = 0.f;         // this warp's share of the previous written row's squared norm
    int64_t r_prev = 0;
    bool wg_prev = false;

    const int grp = warp / kGW;                  // this warp's group: chunks j % kG == grp
    const int gt = tid - grp * kGT;              // thread index inside the group
    const uint32_t toff = (uint32_t)gt * 16u;    // first of this thread's kP pieces in a chunk
    // this thread's tensor-memory window: its lane, 128 of the 512 columns
    const uint32_t tm_lane = TM ? ctrl.tmem_base + ((uint32_t)((warp & 3) * 32) << 16) +
                                      (uint32_t)((warp >> 2) * kTmColsPerThread)
                                : 0u;
    const int64_t iters = my_rows > 0 ? my_rows + 1 : 0;   // + one exchange for the last norm
    Acc2 a;        // sweep-1 sums; carries the leading chunks of the next row across sweep 2
    a.reset();
    for (int64_t i = 0; i < iters; ++i) {
      const bool real = i < my_rows;
      // this row's metadata (the flush iteration has none)
      int64_t rC = 0;
      int yC = 0;
      float zyC = 0.f, uyC = 0.f;
      bool wgC = false;
      if (real) {
        const int ms = (int)(i % kMetaDepth);
        if (!bounded_wait<false>(smem_u32(&ctrl.meta_full[ms]),
                                 (uint32_t)((i / kMetaDepth) & 1), abort, plan.wait_limit_ns)) {
          timed_out = true;
          break;
        }
        const RowMeta& m = ctrl.meta[ms];
        rC = m.r;
        yC = m.y;
        wgC = m.wg != 0;
        zyC = m.zy;
        uyC = m.uy;
      }
      const bool y_valid = (yC >= 0) && ((int64_t)yC < p.V);
      const float ref_s = zyC * kLog2e, ref_t = uyC * kLog2e;   // shared references of the row
      const float dref = wgC ? 0.f : zyC - uyC;                 // delta is centred on probe rows
      const uint32_t rpar = (uint32_t)(i & 1);                  // fill parity of resident slots

      // ---------------------------------------------------------------- sweep 1
      // Visits v in [v0, nch) are chunks of row i (its leading chunks were taken one iteration
      // earlier); at v == nch the row's record is posted to every CTA; visits v in (nch, vend)
      // are the leading streamed chunks of row i+1, taken while the exchange is in flight.
      const int par = (int)(i & 1);
      {
        const int v0 = real ? (i == 0 ? 0 : plan.lead) : nch;
        const int vend = (real && i + 1 < my_rows) ? nch + plan.lead : nch;
        bool wgv = wgC;
        f2_t nrefs = splat2(-ref_s), nreft = splat2(-ref_t), ndref = splat2(-dref);
        for (int v = v0;; ++v) {
          if (v == nch) {
            if (TM) tm_wait_st();
            // record = { S, A, St, B0, B1, B2, q_prev, 0 }: this warp's sums over its lanes.
            const float v0s = lane_sum(hsum2(a.S)), v1 = lane_sum(hsum2(a.A)), v2 = lane_sum(hsum2(a.St));
            float v3 = 0.f, v4 = 0.f, v5 = 0.f;
            if (real && !wgC) {
              v3 = lane_sum(hsum2(a.B0));
              v4 = lane_sum(hsum2(a.B1));
              v5 = lane_sum(hsum2(a.B2));
            }
            if (lane < cl && ADWIN_CHK((int)rank * kNW + warp < kMaxRec && cl <= kMaxCL, p.status)) {
              const uint32_t dst =
                  map_to_rank(smem_u32(&ctrl.xbuf[par][rank * kNW + warp][0]), (uint32_t)lane);
              remote_store4(dst, v0s, v1, v2, v3);
              remote_store4(dst + 16, v4, v5, q_prev, 0.f);
              remote_arrive_release(map_to_rank(smem_u32(&ctrl.xbar[par]), (uint32_t)lane));
            }
            a.reset();
            if (nch >= vend) break;
            // from here on: row i+1
            const int msn = (int)((i + 1) % kMetaDepth);
            if (!bounded_wait<false>(smem_u32(&ctrl.meta_full[msn]),
                                     (uint32_t)(((i + 1) / kMetaDepth) & 1), abort, plan.wait_limit_ns)) {
              timed_out = true;
              break;
            }
            const RowMeta& mn = ctrl.meta[msn];
            wgv = mn.wg != 0;
            const float zyN = mn.zy, uyN = mn.uy;
            nrefs = splat2(-zyN * kLog2e);
            nreft = splat2(-uyN * kLog2e);
            ndref = splat2(-(wgv ? 0.f : zyN - uyN));
          }
          if (v >= vend) break;   // (reached only when the leading chunks of row i+1 are done)
          const int j = v < nch ? v : v - nch;
          if (!ADWIN_CHK(j >= 0 && j < nch && j < kMaxChunks && rc_slot >= 0 && rc_slot < nring + (nring == 0), p.status)) {
            timed_out = true;
            break;
          }
          const int k = ctrl.tab[j];
          const char* sl;
          if (k >= 0) {   // resident chunks only occur in the part of row i (v < nch)
            if (!bounded_wait<false>(smem_u32(&ctrl.res_full[k]), rpar, abort, plan.wait_limit_ns)) timed_out = true;
            sl = res_base + (size_t)k * plan.slot_bytes + toff;
          } else {
            if (!bounded_wait<false>(smem_u32(&ctrl.ring_full[rc_slot]), rc_phase, abort, plan.wait_limit_ns)) timed_out = true;
            sl = ring_base + (size_t)rc_slot * plan.slot_bytes + toff;
          }
          if (timed_out) break;
          // The thread's pieces go to registers first and the slot is handed back at once, so
          // the refill is in flight while the arithmetic runs.
          const int np = pieces_in_chunk(j);
          uint4 zr[kP], ur[kP];
#pragma unroll
          for (int h = 0; h < kP; ++h) {
            if (gt + h * kGT < np &&
                ADWIN_CHK(k < nres && toff + (uint32_t)(h * kGT * 16) + 16u <= u_off, p.status)) {
              zr[h] = *reinterpret_cast<const uint4*>(sl + h * kGT * 16);
              ur[h] = *reinterpret_cast<const uint4*>(sl + u_off + h * kGT * 16);
            }
          }
          if (k < 0 || !wgv) {
            __syncwarp();
            if (lane == 0)
              mbar_arrive(smem_u32(k < 0 ? &ctrl.ring_empty[rc_slot] : &ctrl.res_empty[k]));
          }
          if (TM && k < 0 && wgv) {   // park the pieces for sweep 2 (every lane takes part)
            const int o = ctrl.ord[j];
#pragma unroll
            for (int h = 0; h < kP; ++h)
              if (ADWIN_CHK((o * kP + h) * 8 + 8 <= kTmColsPerThread, p.status))
                tm_store8(tm_lane + (uint32_t)((o * kP + h) * 8), zr[h], ur[h]);
          }
#pragma unroll
          for (int h = 0; h < kP; ++h) {
            if (gt + h * kGT < np) {
              f2_t Z[NP], U[NP];
              Pairs<TIn>::make(zr[h], Z);
              Pairs<TIn>::make(ur[h], U);
              if (wgv)
                acc_grad<NP, kPolyPairs<TIn>()>(Z, U, nrefs, nreft, a);
              else
                acc_probe<NP>(Z, U, nrefs, nreft, ndref, a);
            }
          }
          if (k < 0 && ++rc_slot == nring) {   // the ring cursor walks every streamed chunk
            rc_slot = 0;
            rc_phase ^= 1u;
          }
        }
        if (timed_out) break;
      }

      // ---------------------------------------------------------------- exchange
      RowTotals t;
      float qtot;
      {
        if (!bounded_wait<true>(smem_u32(&ctrl.xbar[par]), (uint32_t)((i >> 1) & 1), abort, plan.wait_limit_ns)) {
          timed_out = true;
          break;
        }
        // fixed-order sum of the nrec records (lane = record, then a butterfly)
        float s[7] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int rr = lane; rr < nrec; rr += 32) {
          const float4 x0 = *reinterpret_cast<const float4*>(&ctrl.xbuf[par][rr][0]);
          const float4 x1 = *reinterpret_cast<const float4*>(&ctrl.xbuf[par][rr][4]);
          s[0] += x0.x; s[1] += x0.y; s[2] += x0.z; s[3] += x0.w;
          s[4] += x1.x; s[5] += x1.y; s[6] += x1.z;
        }
        t.M2s = ref_s;
        t.M2t = ref_t;
        t.S = lane_sum(s[0]);
        t.A = lane_sum(s[1]);
        t.St = lane_sum(s[2]);
        t.B0 = t.B1 = t.B2 = 0.f;
        if (real && !wgC) {
          t.B0 = lane_sum(s[3]);
          t.B1 = lane_sum(s[4]);
          t.B2 = lane_sum(s[5]);
        }
        qtot = lane_sum(s[6]);
      }
      if (warp == 0 && lane == 0 && rank == 0 && i > 0 && wg_prev && p.gsq) p.gsq[r_prev] = qtot;
      if (!real) break;

      // ---------------------------------------------------------------- overflow fallback
      // The totals are identical in every warp of the cluster, so this branch is uniform.
      if (!(t.S < kSumLimit) || !(t.St < kSumLimit) || !(t.B0 < kSumLimit)) {
        RowAcc ra;
        ra.reset();
        const char* zrow = static_cast<const char*>(p.student) + ((size_t)rC * p.ld + (size_t)piece0 * N) * sizeof(TIn);
        const char* urow = static_cast<const char*>(p.teacher) + ((size_t)rC * p.ld + (size_t)piece0 * N) * sizeof(TIn);
        for (int64_t pc = tid; pc < my_pieces; pc += kNT) {
          float z[N], u[N];
          const uint4 zv = __ldg(reinterpret_cast<const uint4*>(zrow) + pc);
          const uint4 uv = __ldg(reinterpret_cast<const uint4*>(urow) + pc);
          Elem<TIn>::unpack(zv, z);
          Elem<TIn>::unpack(uv, u);
          acc_piece<N, true>(z, u, dref, ra);
        }
        const float wms = warp_max(ra.m2s), wmt = warp_max(ra.m2t);
        const float fs = (ra.m2s == -INFINITY) ? 0.f : ex2f(ra.m2s - wms);
        const float ft = (ra.m2t == -INFINITY) ? 0.f : ex2f(ra.m2t - wmt);
        const float fs2 = fs * fs;
        const float w1 = lane_sum(ra.S * fs), w2 = lane_sum(ra.A * fs), w3 = lane_sum(ra.B0 * fs2);
        const float w4 = lane_sum(ra.B1 * fs2), w5 = lane_sum(ra.B2 * fs2), w7 = lane_sum(ra.St * ft);
        if (lane < cl) {
          const uint32_t dst = map_to_rank(smem_u32(&ctrl.sbuf[rank * kNW + warp][0]), (uint32_t)lane);
          remote_store4(dst, wms, w1, w2, w3);
          remote_store4(dst + 16, w4, w5, wmt, w7);
          remote_arrive_release(map_to_rank(smem_u32(&ctrl.sbar), (uint32_t)lane));
        }
        if (!bounded_wait<true>(smem_u32(&ctrl.sbar), safe_rounds & 1u, abort, plan.wait_limit_ns)) {
          timed_out = true;
          break;
        }
        ++safe_rounds;
        float ms = -INFINITY, mt = -INFINITY;
        for (int rr = lane; rr < nrec; rr += 32) {
          ms = fmaxf(ms, ctrl.sbuf[rr][0]);
          mt = fmaxf(mt, ctrl.sbuf[rr][6]);
        }
        t.M2s = warp_max(ms);
        t.M2t = warp_max(mt);
        float s[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int rr = lane; rr < nrec; rr += 32) {
          const float* x = ctrl.sbuf[rr];
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
      }

      // ---------------------------------------------------------------- row scalars
      // (the row's metadata slot stays valid until this warp releases it at the end of the row)
      const RowScalars rs = finish_row(t, zyC, uyC, y_valid, dref, p.alpha, p.mode,
                                       p.row_coef ? &ctrl.meta[i % kMetaDepth].w : nullptr);
      if (warp == 0 && lane == 0 && rank == 0) {
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

      // ---------------------------------------------------------------- sweep 2
      q_prev = 0.f;
      if (wgC) {
        const f2_t L2 = splat2(kLog2e), NEG1 = splat2(-1.f);
        const f2_t nM2s = splat2(-t.M2s), nc0 = splat2(-rs.c0), coef2 = splat2(rs.coef);
        // bf16 logits: g = e * (coef*delta - coef*c0) saves one operation per pair; its rounding
        // (relative to coef*delta, not to the difference) is far inside that dtype's tolerance.
        const f2_t ncc0 = splat2(-rs.coef * rs.c0);
        const int64_t ypiece = y_valid ? ((int64_t)yC / N - piece0) : -1;   // slice-relative
        char* gthread = static_cast<char*>(p.grad) +
                        ((size_t)rC * p.ld_grad + (size_t)(piece0 + gt) * N) * sizeof(TOut);
        const size_t gstep = (size_t)plan.chunk_pieces * N * sizeof(TOut);
        f2_t Q = 0ull;
        for (int j = 0; j < nch; ++j) {
          const int k = ctrl.tab[j];
          if (j % kG == grp) {
            const char* sl = nullptr;
            const bool from_tm = TM && k < 0;
            if (k >= 0) {
              sl = res_base + (size_t)k * plan.slot_bytes + toff;   // still there since sweep 1
            } else if (!TM) {
              if (!bounded_wait<false>(smem_u32(&ctrl.ring_full[rc_slot]), rc_phase, abort, plan.wait_limit_ns)) timed_out = true;
              sl = ring_base + (size_t)rc_slot * plan.slot_bytes + toff;
            }
            if (timed_out) break;
            const int np = pieces_in_chunk(j);
            uint4 zr[kP], ur[kP];
            if (from_tm) {   // back from tensor memory (every lane takes part)
              const int o = ctrl.ord[j];
#pragma unroll
              for (int h = 0; h < kP; ++h)
                if (ADWIN_CHK((o * kP + h) * 8 + 8 <= kTmColsPerThread, p.status))
                  tm_load8(tm_lane + (uint32_t)((o * kP + h) * 8), zr[h], ur[h]);
              tm_wait_ld();
            } else {
#pragma unroll
              for (int h = 0; h < kP; ++h) {
                if (gt + h * kGT < np &&
                    ADWIN_CHK(k < nres && rc_slot < nring + (nring == 0) &&
                                  toff + (uint32_t)(h * kGT * 16) + 16u <= u_off, p.status)) {
                  zr[h] = *reinterpret_cast<const uint4*>(sl + h * kGT * 16);
                  ur[h] = *reinterpret_cast<const uint4*>(sl + u_off + h * kGT * 16);
                }
              }
              __syncwarp();
              if (lane == 0)
                mbar_arrive(smem_u32(k < 0 ? &ctrl.ring_empty[rc_slot] : &ctrl.res_empty[k]));
            }
#pragma unroll
            for (int h = 0; h < kP; ++h) {
              if (gt + h * kGT < np) {
                f2_t Z[NP], U[NP], G[NP];
                Pairs<TIn>::make(zr[h], Z);
                Pairs<TIn>::make(ur[h], U);
#pragma unroll
                for (int e = 0; e < NP; ++e) {
                  const f2_t E = ex2_2(fma2(Z[e], L2, nM2s));
                  if (full_mode) {
                    if (sizeof(TIn) == 2) {
                      G[e] = mul2(E, fma2(fma2(U[e], NEG1, Z[e]), coef2, ncc0));
                    } else {
                      const f2_t D = add2(fma2(U[e], NEG1, Z[e]), nc0);
                      G[e] = mul2(E, mul2(D, coef2));
                    }
                  } else {
                    G[e] = mul2(E, coef2);
                  }
                }
                if (!full_mode && (int64_t)j * plan.chunk_pieces + gt + h * kGT == ypiece) {
                  const int e = (int)((int64_t)yC - ((int64_t)yC / N) * N);
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
                // checked flavour: the 16-byte (or 32-byte) store lies inside the row's V entries
                if (ADWIN_CHK((piece0 + (int64_t)j * plan.chunk_pieces + gt + h * kGT + 1) * N <= p.V &&
                                  rC >= 0 && rC < p.B * p.T, p.status))
                  store_pairs<TOut, NP>(gthread + (size_t)j * gstep + (size_t)h * kGT * N * sizeof(TOut), G);
              }
            }
          } else if (k < 0 && !TM) {
            if (!bounded_wait<false>(smem_u32(&ctrl.ring_full[rc_slot]), rc_phase, abort, plan.wait_limit_ns)) {
              timed_out = true;
              break;
            }
            if (lane == 0) mbar_arrive(smem_u32(&ctrl.ring_empty[rc_slot]));
          }
          if (!TM && k < 0 && ++rc_slot == nring) {
            rc_slot = 0;
            rc_phase ^= 1u;
          }
        }
        if (timed_out) break;
        q_prev = lane_sum(hsum2(Q));
      }
      r_prev = rC;
      wg_prev = wgC;
      // done with this row's metadata slot
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl.meta_empty[i % kMetaDepth]));
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
  if (TM) asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster_sync_all();
  if (TM) {
    __syncthreads();   // every consumer of this CTA is done with tensor memory
    if (warp == kProducerWarp) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      tm_dealloc(ctrl.tmem_base);
    }
  }
}

// ---------------------------------------------------------------------------- host side
namespace {

constexpr int kSmemOptin = 232448;   // 227 KB: the per-CTA limit of sm_100
// Streamed chunks are read a second time by sweep 2; the bytes of one round of rows that have to
// survive in L2 until then should stay well inside the cache.
constexpr double kL2BudgetBytes = 32.0 * 1024 * 1024;

// Chunking and the resident / streamed split for one cluster size.
bool plan_for_cluster(int64_t pieces_total, int cl, bool has_grad, StagedPlan& plan) {
  const int64_t slots_bytes = kSmemOptin - kCtrlBytes;
  const int64_t per_rank = (pieces_total + cl - 1) / cl;
  if (per_rank * 16 > (int64_t)1 << 30) return false;
  int64_t nch = (per_rank + kChunkMax - 1) / kChunkMax;
  int64_t chunk_pieces = (per_rank + nch - 1) / nch;
  chunk_pieces = (chunk_pieces + 7) / 8 * 8;   // slots start on 128-byte boundaries
  if (chunk_pieces > kChunkMax) chunk_pieces = kChunkMax;
  nch = (per_rank + chunk_pieces - 1) / chunk_pieces;
  if (nch > kMaxChunks) return false;
  const int64_t slot_bytes = 2 * chunk_pieces * 16;
  const int64_t nslot = slots_bytes / slot_bytes;
  if (nslot < 2) return false;
  int64_t nres = 0, nring = 0;
  int tm = 0;
  if (!has_grad) {
    nring = nslot < kMaxRing ? nslot : kMaxRing;   // nothing is read twice
  } else {
    // About 0.42 of the slice resident balances the HBM reads of the two sweeps (sweep 1 takes
    // ~1.6x as long as sweep 2); the rest of the slots form the ring.
    nres = (nch * 42 + 50) / 100;
    if (nres > kMaxRes) nres = kMaxRes;
    if (nres > nslot - 2) nres = nslot - 2;      // the ring keeps at least two slots in flight
    if (nres < 0) nres = 0;
    nring = nslot - nres;
    if (nring > kMaxRing) nring = kMaxRing;
    if (nres == nch) nring = 0;                    // everything resident: no stream
    // Tensor-memory mode: the streamed chunks are parked in tensor memory between the sweeps
    // (kTmColsPerThread / (kP * 8) chunks fit); only the chunks beyond that stay resident in shared
    // memory and the whole rest of it is a ring that streams from HBM during both sweeps.
    const int64_t stash = kTmColsPerThread / (kP * 8);
    const int64_t nres_tm = nch > stash ? nch - stash : 0;
    if (nres_tm <= nslot - 2 && nres_tm <= kMaxRes && nres_tm < nch) {
      tm = 1;
      nres = nres_tm;
      nring = nslot - nres;
      if (nring > kMaxRing) nring = kMaxRing;
    }
  }
  plan.cl = cl;
  plan.nch = (int)nch;
  plan.nres = (int)nres;
  plan.nring = (int)nring;
  {
    // Sweep 1 of the next row starts on its leading streamed chunks while the exchange of the
    // current row is in flight (at most kLeadMax chunks, and never the whole slice).
    int lead = 0;
    while (lead < kLeadMax && lead + 1 < nch && ((lead + 1) * nres) / nch == (lead * nres) / nch) ++lead;
    if (nring < 2 || tm) lead = 0;   // (tensor-memory mode: the next row's chunks would overwrite this row's)
    plan.lead = lead;
  }
  plan.chunk_pieces = (int)chunk_pieces;
  plan.per_rank_pieces = (int)per_rank;
  plan.slot_bytes = (uint32_t)slot_bytes;
  plan.tm = tm;
  return true;
}

int plan_smem_bytes(const StagedPlan& plan) {
  return kCtrlBytes + (plan.nres + plan.nring) * (int)plan.slot_bytes;
}

template <typename TIn, typename TOut>
cudaError_t max_clusters_for(const StagedPlan& plan, int sm_count, int& max_clusters) {
  auto kernel = plan.tm ? kl_staged_kernel<TIn, TOut, true> : kl_staged_kernel<TIn, TOut, false>;
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

// The cluster size is chosen once per (device, shape class): the one that keeps the most SMs busy
// (cluster sizes that do not divide a GPC's SM count leave SMs idle) among those whose streamed
// bytes fit the L2 budget, else the one with the fewest streamed bytes.
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
    const double streamed = ctas * (double)(plan.nch - plan.nres) * plan.slot_bytes;
    double score = ctas;
    if (has_grad && streamed > kL2BudgetBytes) score *= kL2BudgetBytes / streamed;
    score -= 1e-3 * cl;
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

  auto kernel = plan.tm ? kl_staged_kernel<TIn, TOut, true> : kl_staged_kernel<TIn, TOut, false>;
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
  plan.wait_limit_ns = handshake_wait_limit_ns();
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
