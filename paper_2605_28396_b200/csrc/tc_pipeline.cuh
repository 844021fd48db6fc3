// Building blocks of the tensor-core kernels (sm_100a): TMA tile loads into swizzled shared
// memory, tcgen05.mma with the accumulator in tensor memory, tcgen05.ld for the epilogue, and
// mbarrier waits that give up after a time limit instead of spinning for ever.
//
// Tile shapes are fixed: an MMA tile is 128 rows (M) x 256 columns (N), one k-block is 64 bf16
// (128 bytes, the span of the 128-byte swizzle), one tcgen05.mma covers K = 16.  A shared-memory
// stage holds the A tile (16 KB) and the B tile (32 KB) of one k-block.
//
// Operand layouts in shared memory (what the TMA boxes below produce and the matrix descriptors
// describe):
//   K-major  (the contraction index is contiguous in global memory): one box {64 k, R rows};
//            row r lies at r*128 bytes, 16-byte units XOR-swizzled with (r % 8); 8-row groups are
//            1024 bytes apart (stride byte offset).
//   MN-major (the row/column index of the tile is contiguous in global memory): one box
//            {64 mn, 64 k} per 64 rows/columns of the tile; k-row j lies at j*128 bytes inside the
//            box, boxes are 8192 bytes apart (leading byte offset), 8-k groups 1024 bytes apart.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace adwin {
namespace tc {

constexpr int kBM = 128;            // rows of an MMA tile (TMEM lanes)
constexpr int kBN = 256;            // columns of an MMA tile (TMEM columns of one accumulator)
constexpr int kBK = 64;             // bf16 per k-block (one 128-byte swizzle span)
constexpr int kUmmaK = 16;          // K of one tcgen05.mma (bf16)
constexpr int kStages = 4;
constexpr int kMaxStages = 6;        // barrier arrays are sized for the deepest pipeline in use
constexpr int kABytes = kBM * kBK * 2;            // 16384
constexpr int kBBytes = kBN * kBK * 2;            // 32768
constexpr int kStageBytes = kABytes + kBBytes;    // 49152
constexpr int kBoxBytesMN = 64 * kBK * 2;         // 8192: one {64 mn, 64 k} box
constexpr int kTmemCols = 512;
constexpr int kThreads = 384;       // warp 0: TMA producer, warp 1: MMA issuer, warp 2: TMEM
                                    // allocation, warp 3: idle, warps 4..11: epilogue
constexpr int kEpiWarp0 = 4;
constexpr int kEpiThreads = 256;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s

// Control block at the start of dynamic shared memory; the stages follow at the next 1024-byte
// boundary.
struct Ctrl {
  unsigned long long full[kMaxStages];   // TMA -> MMA: the stage's tiles have landed
  unsigned long long empty[kMaxStages];  // MMA -> TMA: the stage's tiles have been consumed
  unsigned long long acc_full[2];      // MMA -> epilogue: accumulator slot complete
  unsigned long long acc_empty[2];     // epilogue -> MMA: accumulator slot read out
  unsigned long long drain;            // give-up path: all issued MMAs have retired
  uint32_t tmem_base;
  int abort;
};
constexpr int kCtrlBytes = 1024;
constexpr int kSmemBytes = kCtrlBytes + 1024 + kStages * kStageBytes;   // + alignment slack
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint64_t timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// ---------------------------------------------------------------------------- mbarrier
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void bar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool bar_test_wait(uint32_t bar, uint32_t parity) {
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
// Wait for the phase with the given parity to complete.  Returns false when the CTA has given up
// (another role ran out of time) or when this wait itself exceeds the limit, in which case it
// raises the CTA's abort flag.
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity, volatile int* abort,
                                         uint64_t limit_ns = kWaitLimitNs) {
  if (limit_ns < 16) {   // diagnostic setting: a wait that is not satisfied right now runs out
    if (bar_test_wait(bar, parity)) return true;
    *abort = 1;
    return false;
  }
  if (bar_try_wait(bar, parity)) return true;
  if (*abort) return false;
  const uint64_t t0 = timer_ns();
  for (;;) {
    if (timer_ns() - t0 > limit_ns) {
      *abort = 1;
      return false;
    }
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (bar_try_wait(bar, parity)) return true;
    if (*abort) return false;
  }
}
// The same wait for the give-up path itself: it ignores the abort flag (it runs after the flag is
// up) and only stops at the time limit.
__device__ __forceinline__ bool bar_wait_drain(uint32_t bar, uint32_t parity) {
  const uint64_t t0 = timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (bar_try_wait(bar, parity)) return true;
    if (timer_ns() - t0 > kWaitLimitNs) return false;
  }
}

// ---------------------------------------------------------------------------- TMA
// 2-D tiled load: c0 is the coordinate along the contiguous dimension (elements), c1 the row.
// c0 times the element size must be a multiple of 16 bytes (here always a multiple of 64 bf16).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t c0,
                                            int32_t c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_map(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---------------------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane (lane = 32*(warp % 4) + laneid is
// encoded in bits 16.. of taddr by the caller).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------------- MMA
// Shared-memory matrix descriptor (64 bit): start address >> 4 in bits 0..13, leading byte offset
// >> 4 in bits 16..29, stride byte offset >> 4 in bits 32..45, descriptor version 1 in bits
// 46..47, swizzle mode in bits 61..63 (2 = 128-byte swizzle).
__device__ __forceinline__ uint64_t desc_k_major(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) |
         ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(kBoxBytesMN >> 4) << 16) |
         ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Advance of the encoded start address per K = 16 step inside a k-block.
constexpr uint32_t kStepKMajor = (kUmmaK * 2) >> 4;        // 32 bytes along the swizzled row
constexpr uint32_t kStepMNMajor = (kUmmaK * 128) >> 4;     // 16 k-rows of 128 bytes

// Instruction descriptor of tcgen05.mma.kind::f16 for bf16 x bf16 -> fp32, M = 128, N = 256:
// accumulator format fp32 (bits 4..5 = 1), A and B format bf16 (bits 7..9, 10..12 = 1), operand
// majors in bits 15 / 16 (0 = K-major, 1 = MN-major), N >> 3 in bits 17..22, M >> 4 in bits 24..28.
__host__ __device__ constexpr uint32_t instr_desc(bool a_mn, bool b_mn, int n = kBN) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                     uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on an mbarrier once every tcgen05.mma issued so far by this thread has retired.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   bar)
               : "memory");
}

// The four MMAs of one k-block.  `first` clears the accumulator on the very first MMA of a tile.
template <bool A_MN, bool B_MN, int N = kBN>
__device__ __forceinline__ void issue_kblock(uint32_t tmem_d, uint32_t a_saddr, uint32_t b_saddr,
                                             bool first) {
  constexpr uint32_t idesc = instr_desc(A_MN, B_MN, N);
  const uint64_t ad = A_MN ? desc_mn_major(a_saddr) : desc_k_major(a_saddr);
  const uint64_t bd = B_MN ? desc_mn_major(b_saddr) : desc_k_major(b_saddr);
#pragma unroll
  for (int k = 0; k < kBK / kUmmaK; ++k) {
    umma(tmem_d, ad + (uint64_t)(k * (A_MN ? kStepMNMajor : kStepKMajor)),
         bd + (uint64_t)(k * (B_MN ? kStepMNMajor : kStepKMajor)), idesc,
         (first && k == 0) ? 0u : 1u);
  }
}

// One stage's TMA loads.  Coordinates: (k0, row0) for a K-major operand; (mn0, k0) for an MN-major
// one, where the tile is fetched as 64-wide boxes.
template <bool MN, int ROWS>
__device__ __forceinline__ void load_operand(uint32_t dst, const CUtensorMap* map, int32_t mn0,
                                             int32_t k0, uint32_t bar) {
  if (!MN) {
    tma_load_2d(dst, map, k0, mn0, bar);
  } else {
#pragma unroll
    for (int i = 0; i < ROWS / 64; ++i) tma_load_2d(dst + i * kBoxBytesMN, map, mn0 + 64 * i, k0, bar);
  }
}

// ---------------------------------------------------------------------------- CTA pairs
// Forms used when two CTAs of a cluster work as one MMA unit (cta_group::2): an MMA tile is then
// 256 rows (128 per CTA, each CTA's rows accumulate in its own tensor memory) x 256 columns, and
// each CTA stages only half of the B tile, so the operand bytes per flop that a CTA pulls through
// L2 drop by a third.  The even CTA of the pair (cluster rank 0) issues the MMAs; TMA loads of both
// CTAs report their bytes to its `full` barrier; tcgen05.commit signals barriers at the same
// shared-memory offset in both CTAs.  No load is multicast: each CTA fetches its own tiles.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::
                   : "memory");
}
__device__ __forceinline__ void bar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr)
               : "memory");
}
__device__ __forceinline__ void store_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
// TMA load of a CTA of a pair; `bar_cluster` is the shared::cluster address of the barrier that
// receives the bytes (the even CTA's).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int32_t c0,
                                                 int32_t c1, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void umma_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on the barrier at this shared-memory offset in both CTAs of the pair once every
// tcgen05.mma issued so far has retired.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 "
      "[%0], %1;" ::"r"(bar),
      "h"(mask)
      : "memory");
}
// The four MMAs of one k-block of a pair tile (K-major operands, M = 256).
template <int N>
__device__ __forceinline__ void issue_kblock_pair(uint32_t tmem_d, uint32_t a_saddr,
                                                  uint32_t b_saddr, bool first) {
  constexpr uint32_t idesc = (instr_desc(false, false, N) & ~(0x1fu << 24)) | ((256u >> 4) << 24);
  const uint64_t ad = desc_k_major(a_saddr), bd = desc_k_major(b_saddr);
#pragma unroll
  for (int k = 0; k < kBK / kUmmaK; ++k)
    umma_pair(tmem_d, ad + (uint64_t)(k * kStepKMajor), bd + (uint64_t)(k * kStepKMajor), idesc,
              (first && k == 0) ? 0u : 1u);
}

}  // namespace tc
}  // namespace adwin
