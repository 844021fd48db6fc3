// Fused LM-head form of the windowed OPD divergence: the two policies of Eq. 2 are given as hidden
// states times an output embedding, z = H_s W_s^T and u = H_t W_t^T, and the logits are never
// written to memory.
//
//   plan      tile table over the processed positions (128 consecutive positions of one sequence
//             per tile), compact zero-padded copies of the hidden states
//   sweep 1   per (tile, vocabulary group): 128 x 256 logit tiles of both policies from tcgen05.mma
//             into tensor memory, read back with tcgen05.ld and folded into online log-sum-exp /
//             KL / squared-norm moments; one partial record per (row, group, column half)
//   merge     partial records -> per-token kl, logratio, gsq, lse (float64 combination) and the
//             per-row coefficients of the gradient
//   sweep 2   the same tiles again; the epilogue turns them into the logit gradient
//             G = alpha p (d - KL)  or  alpha c (e_y - p)  (Eq. 2 / Eq. 4) in bf16
//   dH, dW    dH_s = G W_s and dW_s = G^T H_s as two tensor-core GEMMs over G
//
// Every kernel here is persistent (one CTA per SM, static round-robin over work items) and warp
// specialised: warp 0 issues the TMA loads, warp 1 the MMAs, warps 4..11 run the epilogue.
#include <cuda_bf16.h>

#include <mutex>

#include "adwin_common.cuh"
#include "adwin_internal.h"
#include "tc_pipeline.cuh"

namespace adwin {
namespace {

using namespace tc;

constexpr int kRecFields = 8;    // m2s, S, A, B0, B1, B2, m2t, St
constexpr int kTokFields = 4;    // z_y, u_y, has_y, unused
constexpr int kInfoFields = 8;   // L2s, a1, a0, gy, y (bits), unused x3
constexpr int kTileFields = 8;   // b, t0, nvalid, ngrad, gidx, unused x3
// Logit value given to the columns past the vocabulary in the last tile: far enough below any
// real logit that its exponential is exactly zero against a real row maximum, and small enough
// that the rounding residual of z*log2e against the running reference stays a fraction of one
// (a partial that sees only such columns keeps finite sums and merges with weight 2^-huge = 0).
constexpr float kMasked = -1.0e6f;

// ---------------------------------------------------------------------------- workspace
struct LmLayout {
  size_t off_rowmap, off_hdr, off_tiles, off_g2t, off_rowdst, off_info, off_tok, off_part, off_hs,
      off_ht, off_hg, off_G, total;
  int64_t max_tiles;
  int n_groups, n_chunks;
  int64_t ldG;
};

int64_t max_tiles_for(int64_t B, int64_t T, int64_t max_rows) {
  const int64_t per_seq = (T + kBM - 1) / kBM;
  int64_t cap = B * per_seq;
  if (max_rows > 0 && max_rows < B * T) {
    const int64_t bound = (max_rows + kBM - 1) / kBM + B;   // one ragged tile per sequence
    if (bound < cap) cap = bound;
  }
  return cap < 1 ? 1 : cap;
}

LmLayout lm_layout(int64_t B, int64_t T, int64_t V, int64_t ds, int64_t dt, int64_t max_rows,
                   bool want_grad, bool range_full) {
  auto up = [](size_t x) { return (x + 1023) & ~size_t(1023); };
  LmLayout L;
  L.max_tiles = max_tiles_for(B, T, max_rows);
  L.n_chunks = (int)((V + kBN - 1) / kBN);
  L.n_groups = L.n_chunks < 8 ? L.n_chunks : 8;
  L.ldG = (V + 7) / 8 * 8;
  const size_t rows = (size_t)L.max_tiles * kBM;
  size_t o = 0;
  L.off_rowmap = o;  o = up(o + workspace_layout(B).total_ext);
  L.off_hdr = o;     o = up(o + 256);
  L.off_tiles = o;   o = up(o + (size_t)L.max_tiles * kTileFields * 4);
  L.off_g2t = o;     o = up(o + (size_t)L.max_tiles * 4);
  L.off_rowdst = o;  o = up(o + rows * 4);
  L.off_info = o;    o = up(o + rows * kInfoFields * 4);
  L.off_tok = o;     o = up(o + rows * kTokFields * 4);
  L.off_part = o;    o = up(o + rows * (size_t)L.n_groups * 2 * kRecFields * 4);
  L.off_hs = o;      o = up(o + rows * (size_t)ds * 2);
  L.off_ht = o;      o = up(o + rows * (size_t)dt * 2);
  L.off_hg = o;      if (want_grad && range_full) o = up(o + rows * (size_t)ds * 2);
  L.off_G = o;       if (want_grad) o = up(o + rows * (size_t)L.ldG * 2);
  L.total = o;
  return L;
}

// ---------------------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
  static std::mutex mu;
  static EncodeTiledFn fn = nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
            cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 matrix [rows, cols], row pitch in elements; boxes of 64 columns x box_rows rows with the
// 128-byte swizzle; out-of-range elements read as zero.
bool make_map(CUtensorMap* m, const void* base, int64_t cols, int64_t rows, int64_t pitch,
              int box_rows) {
  EncodeTiledFn fn = encode_tiled();
  if (!fn || rows < 1 || cols < 1) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---------------------------------------------------------------------------- plan kernels
// hdr[0] = number of tiles, hdr[1] = number of tiles that hold gradient rows.
__global__ void __launch_bounds__(1024) lm_plan_kernel(const int32_t* __restrict__ range,
                                                       const int32_t* __restrict__ ewin, int64_t B,
                                                       int64_t T, int64_t max_tiles, int32_t* hdr,
                                                       int32_t* tiles, int32_t* g2t,
                                                       int32_t* rowdst, int32_t* status) {
  __shared__ int64_t s_tiles;
  if (threadIdx.x == 0) {
    int64_t nt = 0, ng = 0;
    for (int64_t b = 0; b < B; ++b) {
      nt += (range[b] + kBM - 1) / kBM;
      ng += (ewin[b] + kBM - 1) / kBM;
    }
    if (nt > max_tiles) {   // more processed rows than the workspace was sized for
      atomicOr(status, ADWIN_DEV_WORKSPACE);
      nt = 0;
      ng = 0;
    }
    s_tiles = nt;
    hdr[0] = (int32_t)nt;
    hdr[1] = (int32_t)ng;
  }
  __syncthreads();
  if (s_tiles == 0) return;
  // every thread walks the sequences it owns; the running tile counts are recomputed per thread
  for (int64_t b = threadIdx.x; b < B; b += blockDim.x) {
    int64_t tile = 0, gt = 0;
    for (int64_t c = 0; c < b; ++c) {
      tile += (range[c] + kBM - 1) / kBM;
      gt += (ewin[c] + kBM - 1) / kBM;
    }
    const int P = range[b], E = ewin[b];
    for (int t0 = 0; t0 < P; t0 += kBM, ++tile) {
      const int nvalid = P - t0 < kBM ? P - t0 : kBM;
      int ngrad = E - t0;
      ngrad = ngrad < 0 ? 0 : (ngrad > kBM ? kBM : ngrad);
      if (!ADWIN_CHK(tile < max_tiles && gt < max_tiles, status)) break;
      int32_t* e = tiles + tile * kTileFields;
      e[0] = (int32_t)b;
      e[1] = t0;
      e[2] = nvalid;
      e[3] = ngrad;
      e[4] = ngrad > 0 ? (int32_t)gt : -1;
      if (ngrad > 0) {
        g2t[gt] = (int32_t)tile;
        for (int i = 0; i < kBM; ++i)
          rowdst[gt * kBM + i] = i < ngrad ? (int32_t)(b * T + t0 + i) : -1;
        ++gt;
      }
    }
  }
}

// Compact, zero-padded copy of the hidden states of the processed positions: row tile*128+i of
// dst is src[b, t0+i, :] for i < nvalid and zero otherwise.  by_gtile selects the gradient tiles.
__global__ void __launch_bounds__(256) lm_gather_kernel(const __nv_bfloat16* __restrict__ src,
                                                        int64_t T, int64_t d, const int32_t* hdr,
                                                        const int32_t* __restrict__ tiles,
                                                        const int32_t* __restrict__ g2t,
                                                        bool by_gtile, __nv_bfloat16* dst) {
  const int64_t n_rows = (int64_t)hdr[by_gtile ? 1 : 0] * kBM;
  const int64_t vec_per_row = d / 8;
  for (int64_t row = blockIdx.x; row < n_rows; row += gridDim.x) {
    const int64_t tl = row / kBM;
    const int i = (int)(row % kBM);
    const int32_t* e = tiles + (by_gtile ? g2t[tl] : tl) * kTileFields;
    const int lim = by_gtile ? e[3] : e[2];
    uint4* o = reinterpret_cast<uint4*>(dst + row * d);
    if (i < lim) {
      const uint4* s = reinterpret_cast<const uint4*>(src + ((int64_t)e[0] * T + e[1] + i) * d);
      for (int64_t v = threadIdx.x; v < vec_per_row; v += blockDim.x) o[v] = s[v];
    } else {
      for (int64_t v = threadIdx.x; v < vec_per_row; v += blockDim.x) o[v] = make_uint4(0, 0, 0, 0);
    }
  }
}

// The two logits at the sampled token of every processed position, z_y = h_s . W_s[y] and
// u_y = h_t . W_t[y], as plain fp32 dot products (one warp per compact row).  They give the
// sampled-token log-ratio of Section 2.3 without a search through the logit tiles, and their
// difference is the value the sweep centres z - u on: on a peaked row the sampled token is almost
// surely the peak, where the centred difference is then exactly zero, which keeps the
// single-sweep squared-norm moments well conditioned.
__device__ __forceinline__ float warp_dot_bf16(const __nv_bfloat16* a, const __nv_bfloat16* b,
                                               int64_t d, int lane) {
  float acc = 0.f;
  for (int64_t v = lane; v < d / 8; v += 32) {
    const uint4 x = reinterpret_cast<const uint4*>(a)[v], y = reinterpret_cast<const uint4*>(b)[v];
    float xf[8], yf[8];
    Elem<__nv_bfloat16>::unpack(x, xf);
    Elem<__nv_bfloat16>::unpack(y, yf);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc = fmaf(xf[i], yf[i], acc);
  }
  return warp_sum(acc);
}

__global__ void __launch_bounds__(256) lm_token_kernel(
    const __nv_bfloat16* __restrict__ hs_c, const __nv_bfloat16* __restrict__ ws,
    const __nv_bfloat16* __restrict__ ht_c, const __nv_bfloat16* __restrict__ wt, int64_t T,
    int64_t V, int64_t ds, int64_t dt, const int32_t* hdr, const int32_t* __restrict__ tiles,
    const int32_t* __restrict__ tokens, float* tok) {
  const int lane = threadIdx.x & 31;
  const int64_t n_rows = (int64_t)hdr[0] * kBM;
  for (int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); row < n_rows;
       row += (int64_t)gridDim.x * 8) {
    const int32_t* e = tiles + (row / kBM) * kTileFields;
    const int i = (int)(row % kBM);
    float zy = 0.f, uy = 0.f, has = 0.f;
    if (i < e[2]) {
      const int y = tokens[(int64_t)e[0] * T + e[1] + i];
      if (y >= 0 && y < V) {
        zy = warp_dot_bf16(hs_c + row * ds, ws + (int64_t)y * ds, ds, lane);
        uy = warp_dot_bf16(ht_c + row * dt, wt + (int64_t)y * dt, dt, lane);
        has = 1.f;
      }
    }
    if (lane == 0) {
      float* o = tok + row * kTokFields;
      o[0] = zy;
      o[1] = uy;
      o[2] = has;
      o[3] = 0.f;
    }
  }
}

// ---------------------------------------------------------------------------- sweep kernel
struct SweepParams {
  const int32_t* hdr;
  const int32_t* tiles;
  const int32_t* g2t;
  const float* tok;             // sweep 1 in: z_y, u_y per compact row
  int64_t T, V;
  int ks_blocks, kt_blocks;     // k-blocks of the student / teacher contraction
  int n_chunks, n_groups;
  float* part;                  // sweep 1 out: partial records; sweep 2 out: partial sum g^2
  const float* info;            // sweep 2 in
  __nv_bfloat16* G;             // sweep 2 out
  int64_t ldG;
  int64_t max_tiles;            // capacity of the per-tile buffers (checked flavour)
  uint64_t limit_ns;            // limit of the handshake waits
  int32_t* status;
};

// chunk range of vocabulary group g
__device__ __forceinline__ void group_chunks(const SweepParams& p, int g, int& c0, int& c1) {
  const int per = (p.n_chunks + p.n_groups - 1) / p.n_groups;
  c0 = g * per;
  c1 = c0 + per < p.n_chunks ? c0 + per : p.n_chunks;
  if (c0 > c1) c0 = c1;
}

// MOMENTS = false drops the squared-norm moments from sweep 1 (when every processed row gets its
// gsq from sweep 2, or no gsq is asked for).
// GRAD = false: sweep 1 (statistics).  GRAD = true: sweep 2 (logit gradient); NEED_U = false
// skips the teacher product there (the sampled-token estimator of Eq. 4 does not need it).
template <bool GRAD, bool NEED_U, int BN, bool MOMENTS = true, bool PAIR = false>
__global__ void __launch_bounds__(kThreads, 1)
lm_sweep_kernel(const __grid_constant__ CUtensorMap map_hs, const __grid_constant__ CUtensorMap map_ws,
                const __grid_constant__ CUtensorMap map_ht, const __grid_constant__ CUtensorMap map_wt,
                const SweepParams p) {
  // BN = 256: one accumulator pair (student + teacher tile) fills the 512 TMEM columns, the
  // epilogue and the MMAs of the next chunk alternate.  BN = 128: two pairs, so the epilogue of a
  // chunk overlaps the MMAs of the next, at 1.5x the operand bytes per flop.
  // PAIR: two CTAs of a cluster form one MMA unit (cta_group::2): a 256-row tile pair, each CTA
  // stages its own A tile and half of the B tile (32 KB per stage instead of 48) and reads its own
  // 128 rows of the accumulators; the even CTA issues the MMAs.
  static_assert(!PAIR || BN == 256, "the pair form uses 256-column tiles");
  constexpr int kBrows = PAIR ? BN / 2 : BN;        // rows of the B tile this CTA stages
  constexpr int kStB = kABytes + kBrows * kBK * 2;  // bytes per stage
  constexpr int kSt = (kStages * kStageBytes) / kStB < kMaxStages ? (kStages * kStageBytes) / kStB
                                                                  : kMaxStages;   // pipeline stages
  constexpr int kAcc = kTmemCols / (2 * BN);        // accumulator pairs
  constexpr int kHalf = BN / 2;                     // columns per epilogue warpgroup
  static_assert(kSt <= kMaxStages && kSt * kStB <= kStages * kStageBytes, "stage budget");
  extern __shared__ uint8_t smem_raw[];
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw);
  const uint32_t stage0 = (smem_addr(smem_raw) + kCtrlBytes + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort = &ctrl->abort;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;   // 0: the CTA that issues the MMAs

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSt; ++s) {
      bar_init(smem_addr(&ctrl->full[s]), 1);
      bar_init(smem_addr(&ctrl->empty[s]), 1);
    }
    for (int s = 0; s < kAcc; ++s) {
      bar_init(smem_addr(&ctrl->acc_full[s]), 1);
      bar_init(smem_addr(&ctrl->acc_empty[s]), PAIR ? 2 * (kEpiThreads / 32) : kEpiThreads);
    }
    bar_init(smem_addr(&ctrl->drain), 1);
    ctrl->abort = 0;
    bar_init_fence();
  }
  if (warp == 2) {
    if (PAIR) {
      tmem_alloc_pair(smem_addr(&ctrl->tmem_base), kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_addr(&ctrl->tmem_base), kTmemCols);
      tmem_relinquish();
    }
    tc_fence_before_sync();
  }
  __syncthreads();
  if (PAIR) cluster_sync();   // the partner's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = ctrl->tmem_base;

  // Work items: (tile, vocabulary group), or (pair of consecutive tiles, group) for a CTA pair,
  // in which CTA `rank` owns tile 2*pair + rank (the second tile of the last pair may not exist).
  const int n_tiles = p.hdr[GRAD ? 1 : 0];
  const int64_t n_units = PAIR ? (n_tiles + 1) / 2 : n_tiles;
  const int64_t n_items = n_units * p.n_groups;
  const int64_t first_item = PAIR ? blockIdx.x / 2 : blockIdx.x;
  const int64_t item_step = PAIR ? gridDim.x / 2 : gridDim.x;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int64_t item = first_item; ok && item < n_items; item += item_step) {
        const int tile = (PAIR ? 2 : 1) * (int)(item / p.n_groups) + (int)rank;
        const int g = (int)(item % p.n_groups);
        const int row0 = tile * kBM;          // compact row of the tile (tile or gradient-tile order)
        int c0, c1;
        group_chunks(p, g, c0, c1);
        for (int c = c0; ok && c < c1; ++c) {
          for (int pass = 0; ok && pass < (NEED_U ? 2 : 1); ++pass) {
            const CUtensorMap* ma = pass ? &map_ht : &map_hs;
            const CUtensorMap* mb = pass ? &map_wt : &map_ws;
            const int nk = pass ? p.kt_blocks : p.ks_blocks;
            for (int kb = 0; kb < nk; ++kb, ++it) {
              const uint32_t s = it % kSt, ph = (it / kSt) & 1;
              if (!bar_wait(smem_addr(&ctrl->empty[s]), ph ^ 1, abort, p.limit_ns)) { ok = false; break; }
              const uint32_t bar = smem_addr(&ctrl->full[s]);
              const uint32_t a = stage0 + s * kStB, b = a + kABytes;
              if (PAIR) {
                // both CTAs' bytes are counted by the even CTA's barrier
                if (rank == 0) bar_expect_tx(bar, 2 * kStB);
                const uint32_t bar0 = map_to_cta(bar, 0);
                tma_load_2d_pair(a, ma, kb * kBK, row0, bar0);
                tma_load_2d_pair(b, mb, kb * kBK, c * BN + (int)rank * kBrows, bar0);
              } else {
                bar_expect_tx(bar, kStB);
                tma_load_2d(a, ma, kb * kBK, row0, bar);
                tma_load_2d(b, mb, kb * kBK, c * BN, bar);
              }
            }
          }
        }
      }
      // give up: let the copies in flight land before the CTA's shared memory goes (in a pair the
      // even CTA's barriers count both CTAs' copies, and the final cluster barrier holds the odd
      // CTA until the even one has waited for them)
      if (!ok && rank == 0) {
        const uint32_t n_out = it < (uint32_t)kSt ? it : (uint32_t)kSt;
        for (uint32_t j = it - n_out; j < it; ++j)
          bar_wait_drain(smem_addr(&ctrl->full[j % kSt]), (j / kSt) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      uint32_t it = 0, acc_it = 0;
      bool ok = true;
      for (int64_t item = first_item; ok && item < n_items; item += item_step) {
        int c0, c1;
        group_chunks(p, (int)(item % p.n_groups), c0, c1);
        for (int c = c0; ok && c < c1; ++c, ++acc_it) {
          const uint32_t slot = acc_it % kAcc, aph = (acc_it / kAcc) & 1;
          if (!bar_wait(smem_addr(&ctrl->acc_empty[slot]), aph ^ 1, abort, p.limit_ns)) { ok = false; break; }
          tc_fence_after_sync();
          for (int pass = 0; ok && pass < (NEED_U ? 2 : 1); ++pass) {
            const int nk = pass ? p.kt_blocks : p.ks_blocks;
            const uint32_t tmem_d = tmem_base + slot * (2 * BN) + (pass ? BN : 0);
            for (int kb = 0; kb < nk; ++kb, ++it) {
              const uint32_t s = it % kSt, ph = (it / kSt) & 1;
              if (!bar_wait(smem_addr(&ctrl->full[s]), ph, abort, p.limit_ns)) { ok = false; break; }
              tc_fence_after_sync();
              const uint32_t a = stage0 + s * kStB, b = a + kABytes;
              if (PAIR) {
                issue_kblock_pair<BN>(tmem_d, a, b, kb == 0);
                umma_commit_pair(smem_addr(&ctrl->empty[s]));
              } else {
                issue_kblock<false, false, BN>(tmem_d, a, b, kb == 0);
                umma_commit(smem_addr(&ctrl->empty[s]));
              }
            }
          }
          if (ok) {
            if (PAIR) umma_commit_pair(smem_addr(&ctrl->acc_full[slot]));
            else umma_commit(smem_addr(&ctrl->acc_full[slot]));
          }
        }
      }
      if (!ok) {   // give up: wait until the MMAs already issued have retired
        if (PAIR) umma_commit_pair(smem_addr(&ctrl->drain));
        else umma_commit(smem_addr(&ctrl->drain));
        bar_wait_drain(smem_addr(&ctrl->drain), 0);
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ------------------------------------------------------------------ epilogue
    const int ew = warp - kEpiWarp0;
    const int quad = warp & 3;               // TMEM lanes 32*quad .. 32*quad+31
    const int half = ew >> 2;                // columns half*128 .. half*128+127 of the tile
    const int row = quad * 32 + lane;
    const uint32_t t_quad = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * kHalf);
    uint32_t acc_it = 0;
    bool ok = true;
    for (int64_t item = first_item; ok && item < n_items; item += item_step) {
      const int tile_c = (PAIR ? 2 : 1) * (int)(item / p.n_groups) + (int)rank;
      const int g = (int)(item % p.n_groups);
      const bool live = tile_c < n_tiles;     // the last pair's second tile may not exist
      const int tile = !live ? 0 : (GRAD ? p.g2t[tile_c] : tile_c);
      int c0, c1;
      group_chunks(p, g, c0, c1);

      int y = -1;
      RowAcc acc;
      float dref = 0.f, q = 0.f;   // q: this thread's share of the row's sum g^2 (sweep 2)
      float L2s = 0.f, a1 = 0.f, a0 = 0.f, gy = 0.f;
      acc.reset();
      if (!live) {
        // nothing to read: the tile's accumulators hold products of whatever the loads returned
      } else if (!GRAD) {
        const float* tk = p.tok + ((int64_t)tile * kBM + row) * kTokFields;
        dref = tk[0] - tk[1];      // centre of z - u for this row: the sampled token's difference
      } else {
        const float* inf = p.info + ((int64_t)tile * kBM + row) * kInfoFields;
        L2s = inf[0];
        a1 = inf[1];
        a0 = inf[2];
        gy = inf[3];
        y = __float_as_int(inf[4]);
      }
      for (int c = c0; ok && c < c1; ++c, ++acc_it) {
        const uint32_t slot = acc_it % kAcc, aph = (acc_it / kAcc) & 1;
        const uint32_t t_lane = t_quad + slot * (2 * BN);
        if (!__all_sync(0xffffffffu, bar_wait(smem_addr(&ctrl->acc_full[slot]), aph, abort, p.limit_ns))) {
          ok = false;   // the same decision in every lane: tcgen05.ld below is warp-collective
          break;
        }
        tc_fence_after_sync();
        const int64_t col_base = (int64_t)c * BN + half * kHalf;
        const bool ragged = col_base + kHalf > p.V;
#pragma unroll 1
        for (int j = 0; live && j < kHalf / 32; ++j) {
          uint32_t zr[32], ur[32];
          tmem_ld32(t_lane + j * 32, zr);
          if (NEED_U) tmem_ld32(t_lane + BN + j * 32, ur);
          tmem_ld_wait();
          const int64_t col = col_base + j * 32;
          float z[32], u[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            z[i] = __uint_as_float(zr[i]);
            u[i] = NEED_U ? __uint_as_float(ur[i]) : 0.f;
          }
          if (ragged) {   // columns past the vocabulary: exp -> 0, z - u -> 0
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (col + i >= p.V) {
                z[i] = kMasked;
                u[i] = kMasked;
              }
          }
          if (!GRAD) {
            acc_piece<32, MOMENTS>(z, u, dref, acc);
          } else {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              float gv[2];
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const float pz = ex2f(fmaf(z[i + e], kLog2e, -L2s));
                const float w = NEED_U ? fmaf(a1, z[i + e] - u[i + e], a0) : a0;
                gv[e] = pz * w;
                q = fmaf(gv[e], gv[e], q);
              }
              pk[i >> 1] = pack_bf16x2(gv[0], gv[1]);
            }
            if ((unsigned)(y - (int)col) < 32u) {   // the sampled token's own entry (Eq. 4)
              const int yi = y - (int)col;
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (i == yi) {
                  const float pz = ex2f(fmaf(z[i], kLog2e, -L2s));
                  const float w = NEED_U ? fmaf(a1, z[i] - u[i], a0) : a0;
                  const float gv = fmaf(pz, w, gy);
                  q += gv * gv - (pz * w) * (pz * w);
                  const uint32_t h = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(gv));
                  pk[i >> 1] = (i & 1) ? ((pk[i >> 1] & 0x0000ffffu) | (h << 16))
                                       : ((pk[i >> 1] & 0xffff0000u) | h);
                }
            }
            __nv_bfloat16* gp = p.G + ((int64_t)tile_c * kBM + row) * p.ldG + col;
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (col + v * 8 < p.V &&
                  ADWIN_CHK(tile_c < p.max_tiles && col + v * 8 + 8 <= p.ldG, p.status))
                *reinterpret_cast<uint4*>(gp + v * 8) =
                    make_uint4(pk[v * 4], pk[v * 4 + 1], pk[v * 4 + 2], pk[v * 4 + 3]);
          }
        }
        tc_fence_before_sync();
        if (PAIR) {   // one arrival per warp: the odd CTA's arrivals cross to the even CTA
          __syncwarp();
          if (lane == 0) {
            if (rank != 0) bar_arrive_cluster(map_to_cta(smem_addr(&ctrl->acc_empty[slot]), 0));
            else bar_arrive(smem_addr(&ctrl->acc_empty[slot]));
          }
        } else {
          bar_arrive(smem_addr(&ctrl->acc_empty[slot]));
        }
      }
      if (GRAD && ok && live && ADWIN_CHK(tile_c < p.max_tiles && g < p.n_groups, p.status))
        p.part[(((int64_t)tile_c * p.n_groups + g) * 2 + half) * kBM + row] = q;
      if (!GRAD && ok && live && ADWIN_CHK(tile < p.max_tiles && g < p.n_groups && row < kBM, p.status)) {
        float* o = p.part + ((((int64_t)tile * p.n_groups + g) * 2 + half) * kRecFields) * kBM + row;
        o[0 * kBM] = acc.m2s;
        o[1 * kBM] = acc.S;
        o[2 * kBM] = acc.A;
        o[3 * kBM] = acc.B0;
        o[4 * kBM] = acc.B1;
        o[5 * kBM] = acc.B2;
        o[6 * kBM] = acc.m2t;
        o[7 * kBM] = acc.St;
      }
    }
  }
  if (*abort && threadIdx.x == 0) {
    atomicOr(p.status, ADWIN_DEV_TIMEOUT);
    if (PAIR) store_cluster_u32(map_to_cta(smem_addr(&ctrl->abort), rank ^ 1u), 1u);   // partner too
  }
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) cluster_sync();   // neither CTA leaves while the other may still use its memory
  if (warp == 2) {
    tc_fence_after_sync();
    if (PAIR) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------- merge kernel
struct MergeParams {
  const int32_t* hdr;
  const int32_t* tiles;
  const int32_t* tokens;
  const float* part;
  const float* tok;
  float* info;
  int64_t T, V;
  int n_groups;
  float alpha;
  int mode;
  float* kl;
  float* logratio;
  float* gsq;
  float* lse_s;
  float* lse_t;
  int32_t* status;
};

// One thread per compact row: combine the partial records of the row in float64 against common
// references and derive the per-token outputs and the gradient coefficients of sweep 2:
//   g_k = p_k (a1 (z_k - u_k) + a0) (+ gy at k = y),   p_k = 2^(z_k log2e - L2s).
__global__ void __launch_bounds__(kBM) lm_merge_kernel(const MergeParams p) {
  const int tile = blockIdx.x;
  if (tile >= p.hdr[0]) return;
  const int row = threadIdx.x;
  const int32_t* te = p.tiles + (int64_t)tile * kTileFields;
  float* inf = p.info + ((int64_t)tile * kBM + row) * kInfoFields;
  if (row >= te[2]) {
    inf[0] = 0.f; inf[1] = 0.f; inf[2] = 0.f; inf[3] = 0.f; inf[4] = __int_as_float(-1);
    return;
  }
  const int n = p.n_groups * 2;
  const float* rec = p.part + ((int64_t)tile * n * kRecFields) * kBM + row;
  auto f = [&](int i, int k) { return (double)rec[((int64_t)i * kRecFields + k) * kBM]; };
  double M2s = -INFINITY, M2t = -INFINITY;
  for (int i = 0; i < n; ++i) {
    M2s = fmax(M2s, f(i, 0));
    M2t = fmax(M2t, f(i, 6));
  }
  const float* tk = p.tok + ((int64_t)tile * kBM + row) * kTokFields;
  const bool has_y = tk[2] != 0.f;
  const double zy = tk[0], uy = tk[1];
  const double dref = (double)(tk[0] - tk[1]);   // the centre the sweep used (an fp32 difference)
  double S = 0, St = 0, Ac = 0;
  for (int i = 0; i < n; ++i) {
    const double w = exp2(f(i, 0) - M2s);
    S += w * f(i, 1);
    Ac += w * f(i, 2);
    St += exp2(f(i, 6) - M2t) * f(i, 7);
  }
  const double sh = -Ac / S;                   // centre minus E_p[z - u]
  const double c0 = dref - sh;                 // E_p[z - u]
  double B0 = 0, B2c = 0;
  for (int i = 0; i < n; ++i) {
    const double w = exp2(f(i, 0) - M2s), w2 = w * w;
    B0 += w2 * f(i, 3);
    B2c += w2 * (f(i, 5) + 2.0 * sh * f(i, 4) + sh * sh * f(i, 3));
  }
  constexpr double kLn2 = 0.69314718055994530942;
  const double lse_s = (M2s + log2(S)) * kLn2, lse_t = (M2t + log2(St)) * kLn2;
  const double delta = lse_s - lse_t;
  const double kl = c0 - delta;
  const double c = has_y ? (zy - uy) - delta : (double)NAN;
  const double alpha = p.alpha;
  double gsq, a1, a0, gy;
  if (p.mode == ADWIN_GRAD_FULL_KL) {
    gsq = alpha * alpha * fmax(B2c, 0.0) / (S * S);
    a1 = alpha;
    a0 = -alpha * c0;
    gy = 0.0;
  } else {
    const double py = has_y ? exp2(zy * 1.4426950408889634074 - M2s) / S : (double)NAN;
    const double rest = fmax(B0 / (S * S) - py * py, 0.0);
    gsq = alpha * alpha * c * c * ((1.0 - py) * (1.0 - py) + rest);
    a1 = 0.0;
    a0 = -alpha * c;
    gy = alpha * c;
  }
  const int64_t r = (int64_t)te[0] * p.T + te[1] + row;
  p.kl[r] = (float)kl;
  p.logratio[r] = (float)c;
  if (p.gsq) p.gsq[r] = (float)gsq;
  if (p.lse_s) p.lse_s[r] = (float)lse_s;
  if (p.lse_t) p.lse_t[r] = (float)lse_t;
  const bool in_grad = row < te[3];
  inf[0] = in_grad ? (float)(lse_s * 1.4426950408889634074) : 0.f;
  inf[1] = in_grad ? (float)a1 : 0.f;
  inf[2] = in_grad ? (float)a0 : 0.f;
  inf[3] = in_grad ? (float)gy : 0.f;
  inf[4] = __int_as_float(in_grad && has_y ? p.tokens[r] : -1);
  if (!has_y) atomicOr(p.status, ADWIN_DEV_TOKEN_RANGE);
  if (!(isfinite(lse_s) && isfinite(lse_t))) atomicOr(p.status, ADWIN_DEV_NONFINITE);
}

// Squared gradient norm of the rows whose gradient sweep 2 formed: the sum of g_k^2 over the
// entries themselves (fixed order, float64), which replaces the single-sweep moment value there.
__global__ void __launch_bounds__(kBM) lm_gsq_kernel(const int32_t* hdr, const float* __restrict__ part,
                                                     const int32_t* __restrict__ rowdst,
                                                     int n_groups, float* gsq) {
  const int gt = blockIdx.x;
  if (gt >= hdr[1]) return;
  const int row = threadIdx.x;
  const int32_t dst = rowdst[(int64_t)gt * kBM + row];
  if (dst < 0) return;
  double acc = 0.0;
  for (int i = 0; i < n_groups * 2; ++i)
    acc += (double)part[((int64_t)gt * n_groups * 2 + i) * kBM + row];
  gsq[dst] = (float)acc;
}

// ---------------------------------------------------------------------------- GEMM kernel
// C[M,N] = A B with A[m,k], B[n,k] read through TMA in either major, fp32 accumulation in tensor
// memory (two accumulator slots, so the epilogue of a tile overlaps the MMAs of the next one).
struct GemmParams {
  int64_t M, N;                 // extents of C (rows beyond M / columns beyond N are not stored)
  int m_tiles, n_tiles, k_blocks;
  const int32_t* m_tiles_dev;   // optional device-side override of m_tiles (index into hdr)
  const int32_t* k_tiles_dev;   // optional: k_blocks = 2 * (*k_tiles_dev) (128 rows per tile)
  const int32_t* k_list;        // optional: contraction row of every k-block (instead of kb*64)
  const int32_t* k_count_dev;   // with k_list: number of k-blocks
  const int32_t* row_map;       // optional: destination row of every C row, or -1 (skip)
  void* C;
  int64_t ldc;
  int c_is_bf16;
  int32_t* status;
  uint64_t limit_ns;            // limit of the handshake waits
};

template <bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw);
  const uint32_t stage0 = (smem_addr(smem_raw) + kCtrlBytes + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort = &ctrl->abort;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      bar_init(smem_addr(&ctrl->full[s]), 1);
      bar_init(smem_addr(&ctrl->empty[s]), 1);
    }
    for (int s = 0; s < 2; ++s) {
      bar_init(smem_addr(&ctrl->acc_full[s]), 1);
      bar_init(smem_addr(&ctrl->acc_empty[s]), kEpiThreads);
    }
    bar_init(smem_addr(&ctrl->drain), 1);
    ctrl->abort = 0;
    bar_init_fence();
  }
  if (warp == 2) {
    tmem_alloc(smem_addr(&ctrl->tmem_base), kTmemCols);
    tmem_relinquish();
    tc_fence_before_sync();
  }
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = ctrl->tmem_base;

  const int m_tiles = p.m_tiles_dev ? *p.m_tiles_dev : p.m_tiles;
  const int nk = p.k_list ? *p.k_count_dev : (p.k_tiles_dev ? 2 * (*p.k_tiles_dev) : p.k_blocks);
  const int64_t n_items = (int64_t)m_tiles * p.n_tiles;

  if (warp == 0) {
    if (lane == 0 && nk > 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int64_t item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const int m0 = (int)(item / p.n_tiles) * kBM, n0 = (int)(item % p.n_tiles) * kBN;
        for (int kb = 0; kb < nk; ++kb, ++it) {
          const uint32_t s = it % kStages, ph = (it / kStages) & 1;
          if (!bar_wait(smem_addr(&ctrl->empty[s]), ph ^ 1, abort, p.limit_ns)) { ok = false; break; }
          const uint32_t bar = smem_addr(&ctrl->full[s]);
          const uint32_t a = stage0 + s * kStageBytes, b = a + kABytes;
          bar_expect_tx(bar, kStageBytes);
          const int k0 = p.k_list ? p.k_list[kb] : kb * kBK;
          load_operand<A_MN, kBM>(a, &map_a, m0, k0, bar);
          load_operand<B_MN, kBN>(b, &map_b, n0, k0, bar);
        }
      }
      if (!ok) {
        const uint32_t n_out = it < (uint32_t)kStages ? it : (uint32_t)kStages;
        for (uint32_t j = it - n_out; j < it; ++j)
          bar_wait_drain(smem_addr(&ctrl->full[j % kStages]), (j / kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t it = 0, acc_it = 0;
      bool ok = true;
      for (int64_t item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++acc_it) {
        const uint32_t slot = acc_it & 1, aph = (acc_it >> 1) & 1;
        if (!bar_wait(smem_addr(&ctrl->acc_empty[slot]), aph ^ 1, abort, p.limit_ns)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + slot * kBN;
        for (int kb = 0; kb < nk; ++kb, ++it) {
          const uint32_t s = it % kStages, ph = (it / kStages) & 1;
          if (!bar_wait(smem_addr(&ctrl->full[s]), ph, abort, p.limit_ns)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a = stage0 + s * kStageBytes, b = a + kABytes;
          issue_kblock<A_MN, B_MN>(tmem_d, a, b, kb == 0);
          umma_commit(smem_addr(&ctrl->empty[s]));
        }
        if (ok) {
          if (nk > 0) umma_commit(smem_addr(&ctrl->acc_full[slot]));
          else bar_arrive(smem_addr(&ctrl->acc_full[slot]));
        }
      }
      if (!ok) {
        umma_commit(smem_addr(&ctrl->drain));
        bar_wait_drain(smem_addr(&ctrl->drain), 0);
      }
    }
  } else if (warp >= kEpiWarp0) {
    const int ew = warp - kEpiWarp0;
    const int quad = warp & 3, half = ew >> 2;
    const int row = quad * 32 + lane;
    uint32_t acc_it = 0;
    bool ok = true;
    for (int64_t item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++acc_it) {
      const uint32_t slot = acc_it & 1, aph = (acc_it >> 1) & 1;
      const int64_t m = (int64_t)(item / p.n_tiles) * kBM + row;
      const int64_t n0 = (int64_t)(item % p.n_tiles) * kBN + half * 128;
      if (!__all_sync(0xffffffffu, bar_wait(smem_addr(&ctrl->acc_full[slot]), aph, abort, p.limit_ns))) {
        ok = false;
        break;
      }
      tc_fence_after_sync();
      int64_t dst = m;
      if (p.row_map) dst = (m < p.M) ? p.row_map[m] : -1;
      const bool store = m < p.M && dst >= 0 && ADWIN_CHK(n0 >= 0 && n0 < (int64_t)p.n_tiles * kBN, p.status);
      const uint32_t t_lane =
          tmem_base + ((uint32_t)(quad * 32) << 16) + slot * kBN + (uint32_t)(half * 128);
#pragma unroll 1
      for (int j = 0; j < 4; ++j) {
        uint32_t r[32];
        if (nk > 0) {
          tmem_ld32(t_lane + j * 32, r);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0u;
        }
        const int64_t n = n0 + j * 32;
        if (store) {
          if (p.c_is_bf16) {
            __nv_bfloat16* cp = static_cast<__nv_bfloat16*>(p.C) + dst * p.ldc + n;
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (n + v * 8 < p.N)
                *reinterpret_cast<uint4*>(cp + v * 8) = make_uint4(
                    pack_bf16x2(__uint_as_float(r[v * 8]), __uint_as_float(r[v * 8 + 1])),
                    pack_bf16x2(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3])),
                    pack_bf16x2(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5])),
                    pack_bf16x2(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7])));
          } else {
            float* cp = static_cast<float*>(p.C) + dst * p.ldc + n;
#pragma unroll
            for (int v = 0; v < 8; ++v)
              if (n + v * 4 < p.N)
                *reinterpret_cast<uint4*>(cp + v * 4) =
                    make_uint4(r[v * 4], r[v * 4 + 1], r[v * 4 + 2], r[v * 4 + 3]);
          }
        }
      }
      tc_fence_before_sync();
      bar_arrive(smem_addr(&ctrl->acc_empty[slot]));
    }
  }
  if (*abort && threadIdx.x == 0) atomicOr(p.status, ADWIN_DEV_TIMEOUT);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// One sweep launch: single CTAs, or clusters of two for the pair form.
template <bool GRAD, bool NEED_U, int BN, bool MOM, bool PAIR>
cudaError_t launch_sweep(const CUtensorMap& m_hs, const CUtensorMap& m_ws, const CUtensorMap& m_ht,
                         const CUtensorMap& m_wt, const SweepParams& sp, int sm_count,
                         cudaStream_t s) {
  auto kernel = lm_sweep_kernel<GRAD, NEED_U, BN, MOM, PAIR>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(PAIR ? (sm_count & ~1) : sm_count);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = PAIR ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, m_hs, m_ws, m_ht, m_wt, sp);
}

template <typename K>
cudaError_t opt_in_smem(K kernel) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

}  // namespace

// C[M,N] = A B on the tensor cores.  A is [M,K] (K contiguous, a_mn = false) or [K,M] (M
// contiguous, a_mn = true); B is [N,K] or [K,N] likewise; bf16 in, fp32 accumulation.
cudaError_t launch_tc_gemm(const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb,
                           bool b_mn, int64_t M, int64_t N, int64_t K, void* C, int64_t ldc,
                           bool c_bf16, const int32_t* m_tiles_dev, const int32_t* k_tiles_dev,
                           const int32_t* row_map, int32_t* status, int sm_count, cudaStream_t s,
                           const int32_t* k_list, const int32_t* k_count_dev) {
  CUtensorMap ma, mb;
  const bool oka = a_mn ? make_map(&ma, A, M, K, lda, 64) : make_map(&ma, A, K, M, lda, kBM);
  const bool okb = b_mn ? make_map(&mb, B, N, K, ldb, 64) : make_map(&mb, B, K, N, ldb, kBN);
  if (!oka || !okb) return cudaErrorInvalidValue;
  GemmParams p;
  p.M = M;
  p.N = N;
  p.m_tiles = (int)((M + kBM - 1) / kBM);
  p.n_tiles = (int)((N + kBN - 1) / kBN);
  p.k_blocks = (int)((K + kBK - 1) / kBK);
  p.m_tiles_dev = m_tiles_dev;
  p.k_tiles_dev = k_tiles_dev;
  p.k_list = k_list;
  p.k_count_dev = k_count_dev;
  p.row_map = row_map;
  p.C = C;
  p.ldc = ldc;
  p.c_is_bf16 = c_bf16 ? 1 : 0;
  p.status = status;
  p.limit_ns = handshake_wait_limit_ns();
  cudaError_t e;
#define ADWIN_LAUNCH_GEMM(AM, BM_)                                                    \
  do {                                                                                \
    e = opt_in_smem(tc_gemm_kernel<AM, BM_>);                                         \
    if (e != cudaSuccess) return e;                                                   \
    tc_gemm_kernel<AM, BM_><<<sm_count, kThreads, kSmemBytes, s>>>(ma, mb, p);        \
  } while (0)
  if (!a_mn && !b_mn) ADWIN_LAUNCH_GEMM(false, false);
  else if (!a_mn && b_mn) ADWIN_LAUNCH_GEMM(false, true);
  else if (a_mn && !b_mn) ADWIN_LAUNCH_GEMM(true, false);
  else ADWIN_LAUNCH_GEMM(true, true);
#undef ADWIN_LAUNCH_GEMM
  return cudaGetLastError();
}

// Column width of the sweeps' logit tiles.  256 is what the library runs: one accumulator pair
// fills the tensor memory and the epilogue alternates with the MMAs.  The 128-column form (two
// pairs, epilogue overlapped) is correct but measured 1.5x slower at the paper-scale shape -- its
// MMAs are bound by operand traffic -- and is only instantiated in development builds.
#ifdef ADWIN_DEV_EXPORTS
#define ADWIN_SWEEP_128 1
#else
#define ADWIN_SWEEP_128 0
#endif
// CTA pairs (tcgen05 cta_group::2: a 256-row tile pair per MMA, each CTA staging half of the B
// tile).  Correct (the whole test-suite passes with it) and it cuts the operand bytes a CTA pulls
// through L2 by a third, but at the paper-scale shape it measured no faster than single CTAs
// (44.4 ms against 42.2 ms for the statistics sweep): the partner CTAs' epilogues have to meet
// before the next chunk's MMAs start.  Instantiated in development builds only.
static int g_sweep_pair = 0;
void set_sweep_pair(int on) { g_sweep_pair = (ADWIN_SWEEP_128 && on) ? 1 : 0; }
static int g_sweep_bn = 256;
void set_sweep_tile_columns(int bn) { g_sweep_bn = (ADWIN_SWEEP_128 && bn == 128) ? 128 : 256; }

size_t lmhead_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t ds, int64_t dt,
                              int64_t max_rows, bool want_grad, bool range_full) {
  return lm_layout(B, T, V, ds, dt, max_rows, want_grad, range_full).total;
}

// The whole fused pass; arguments validated by the caller.
cudaError_t launch_lmhead(const void* hs, const void* ws, const void* ht, const void* wt, int64_t B,
                          int64_t T, int64_t V, int64_t ds, int64_t dt, const int32_t* tokens,
                          const int32_t* window, const int32_t* rollout_len, float alpha, int mode,
                          int flags, void* dH, int dh_dtype, float* dW, float* kl, float* logratio,
                          float* gsq, float* lse_s, float* lse_t, void* workspace,
                          int64_t max_rows, int32_t* status, int sm_count, cudaStream_t s,
                          bool keep_G) {
  const bool want_grad = dH != nullptr || dW != nullptr || keep_G;
  const bool range_full = (flags & ADWIN_RANGE_FULL) != 0;
  const LmLayout L = lm_layout(B, T, V, ds, dt, max_rows, want_grad, range_full);
  char* wb = static_cast<char*>(workspace);
  int32_t* hdr = reinterpret_cast<int32_t*>(wb + L.off_hdr);
  int32_t* tiles = reinterpret_cast<int32_t*>(wb + L.off_tiles);
  int32_t* g2t = reinterpret_cast<int32_t*>(wb + L.off_g2t);
  int32_t* rowdst = reinterpret_cast<int32_t*>(wb + L.off_rowdst);
  float* info = reinterpret_cast<float*>(wb + L.off_info);
  float* tok = reinterpret_cast<float*>(wb + L.off_tok);
  float* part = reinterpret_cast<float*>(wb + L.off_part);
  __nv_bfloat16* hs_c = reinterpret_cast<__nv_bfloat16*>(wb + L.off_hs);
  __nv_bfloat16* ht_c = reinterpret_cast<__nv_bfloat16*>(wb + L.off_ht);
  __nv_bfloat16* hs_g = range_full ? reinterpret_cast<__nv_bfloat16*>(wb + L.off_hg) : hs_c;
  __nv_bfloat16* G = reinterpret_cast<__nv_bfloat16*>(wb + L.off_G);
  const int64_t rows_cap = L.max_tiles * kBM;

  cudaError_t e = launch_rowmap(window, rollout_len, B, T, flags & ADWIN_RANGE_FULL, wb + L.off_rowmap,
                                false, kl, logratio, gsq, lse_s, lse_t, status, s);
  if (e != cudaSuccess) return e;
  const WorkspaceLayout wl = workspace_layout(B);
  const int32_t* range = reinterpret_cast<const int32_t*>(wb + L.off_rowmap + wl.off_range);
  const int32_t* ewin = reinterpret_cast<const int32_t*>(wb + L.off_rowmap + wl.off_ewin);
  lm_plan_kernel<<<1, 1024, 0, s>>>(range, ewin, B, T, L.max_tiles, hdr, tiles, g2t, rowdst, status);
  const int gather_blocks = (int)(rows_cap < 8192 ? rows_cap : 8192);
  lm_gather_kernel<<<gather_blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(hs), T, ds, hdr,
                                                 tiles, g2t, false, hs_c);
  lm_gather_kernel<<<gather_blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(ht), T, dt, hdr,
                                                 tiles, g2t, false, ht_c);
  if (want_grad && range_full)
    lm_gather_kernel<<<gather_blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(hs), T, ds,
                                                   hdr, tiles, g2t, true, hs_g);
  lm_token_kernel<<<gather_blocks, 256, 0, s>>>(hs_c, static_cast<const __nv_bfloat16*>(ws), ht_c,
                                                static_cast<const __nv_bfloat16*>(wt), T, V, ds, dt,
                                                hdr, tiles, tokens, tok);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;

  const int bn = g_sweep_bn;
  CUtensorMap m_hs, m_ws, m_ht, m_wt;
  if (!make_map(&m_hs, hs_c, ds, rows_cap, ds, kBM) || !make_map(&m_ws, ws, ds, V, ds, bn) ||
      !make_map(&m_ht, ht_c, dt, rows_cap, dt, kBM) || !make_map(&m_wt, wt, dt, V, dt, bn))
    return cudaErrorInvalidValue;

  SweepParams sp;
  sp.hdr = hdr;
  sp.tiles = tiles;
  sp.g2t = g2t;
  sp.tok = tok;
  sp.T = T;
  sp.V = V;
  sp.ks_blocks = (int)((ds + kBK - 1) / kBK);
  sp.kt_blocks = (int)((dt + kBK - 1) / kBK);
  sp.n_chunks = (int)((V + bn - 1) / bn);
  sp.n_groups = L.n_groups;
  sp.part = part;
  sp.info = info;
  sp.G = G;
  sp.ldG = L.ldG;
  sp.max_tiles = L.max_tiles;
  sp.limit_ns = handshake_wait_limit_ns();
  sp.status = status;
  // 128-row boxes of the output embeddings for the pair form (each CTA stages half a B tile)
  const bool pair = ADWIN_SWEEP_128 && g_sweep_pair && bn == 256 && sm_count >= 2;
  CUtensorMap m_ws_h = m_ws, m_wt_h = m_wt;
  if (pair && (!make_map(&m_ws_h, ws, ds, V, ds, kBN / 2) || !make_map(&m_wt_h, wt, dt, V, dt, kBN / 2)))
    return cudaErrorInvalidValue;
  // the single-sweep moments are only needed for rows whose gsq does not come from sweep 2
  const bool moments = gsq != nullptr && (!want_grad || range_full);
  if (bn != 256) {
#if ADWIN_SWEEP_128
    e = launch_sweep<false, true, 128, true, false>(m_hs, m_ws, m_ht, m_wt, sp, sm_count, s);
#endif
#if ADWIN_SWEEP_128
  } else if (pair) {
    e = moments ? launch_sweep<false, true, 256, true, true>(m_hs, m_ws_h, m_ht, m_wt_h, sp, sm_count, s)
                : launch_sweep<false, true, 256, false, true>(m_hs, m_ws_h, m_ht, m_wt_h, sp, sm_count, s);
#endif
  } else {
    e = moments ? launch_sweep<false, true, 256, true, false>(m_hs, m_ws, m_ht, m_wt, sp, sm_count, s)
                : launch_sweep<false, true, 256, false, false>(m_hs, m_ws, m_ht, m_wt, sp, sm_count, s);
  }
  if (e != cudaSuccess) return e;
  if ((e = cudaGetLastError()) != cudaSuccess) return e;

  MergeParams mp;
  mp.hdr = hdr;
  mp.tiles = tiles;
  mp.tokens = tokens;
  mp.part = part;
  mp.tok = tok;
  mp.info = info;
  mp.T = T;
  mp.V = V;
  mp.n_groups = L.n_groups;
  mp.alpha = alpha;
  mp.mode = mode;
  mp.kl = kl;
  mp.logratio = logratio;
  mp.gsq = gsq;
  mp.lse_s = lse_s;
  mp.lse_t = lse_t;
  mp.status = status;
  lm_merge_kernel<<<(unsigned)L.max_tiles, kBM, 0, s>>>(mp);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  if (!want_grad) return cudaSuccess;

  // sweep 2: the gradient tiles' logits again, written out as G (bf16, one row per compact row)
  CUtensorMap m_hg = m_hs;
  if (range_full && !make_map(&m_hg, hs_g, ds, rows_cap, ds, kBM)) return cudaErrorInvalidValue;
  if (mode == ADWIN_GRAD_FULL_KL) {
    // With ADWIN_RANGE_FULL the compact teacher copy is in tile order and sweep 1 is done with it:
    // gather the gradient tiles' rows into the same buffer.
    if (range_full)
      lm_gather_kernel<<<gather_blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(ht), T, dt,
                                                     hdr, tiles, g2t, true, ht_c);
    if (bn != 256) {
#if ADWIN_SWEEP_128
      e = launch_sweep<true, true, 128, true, false>(m_hg, m_ws, m_ht, m_wt, sp, sm_count, s);
#endif
#if ADWIN_SWEEP_128
    } else if (pair) {
      e = launch_sweep<true, true, 256, true, true>(m_hg, m_ws_h, m_ht, m_wt_h, sp, sm_count, s);
#endif
    } else {
      e = launch_sweep<true, true, 256, true, false>(m_hg, m_ws, m_ht, m_wt, sp, sm_count, s);
    }
  } else {
    if (bn != 256) {
#if ADWIN_SWEEP_128
      e = launch_sweep<true, false, 128, true, false>(m_hg, m_ws, m_ht, m_wt, sp, sm_count, s);
#endif
#if ADWIN_SWEEP_128
    } else if (pair) {
      e = launch_sweep<true, false, 256, true, true>(m_hg, m_ws_h, m_ht, m_wt_h, sp, sm_count, s);
#endif
    } else {
      e = launch_sweep<true, false, 256, true, false>(m_hg, m_ws, m_ht, m_wt, sp, sm_count, s);
    }
  }
  if (e != cudaSuccess) return e;
  if (gsq) lm_gsq_kernel<<<(unsigned)L.max_tiles, kBM, 0, s>>>(hdr, part, rowdst, L.n_groups, gsq);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;

  if (dH) {
    if (flags & ADWIN_ZERO_TAIL) {
      e = cudaMemsetAsync(dH, 0, (size_t)B * T * ds * (dh_dtype == ADWIN_F32 ? 4 : 2), s);
      if (e != cudaSuccess) return e;
    }
    // dH_s[rows, d_s] = G[rows, V] W_s[V, d_s]: A K-major, B MN-major; rows scattered to [B,T]
    e = launch_tc_gemm(G, L.ldG, false, ws, ds, true, rows_cap, ds, V, dH, ds,
                       dh_dtype == ADWIN_BF16, hdr + 1, nullptr, rowdst, status, sm_count, s);
    if (e != cudaSuccess) return e;
  }
  if (dW) {
    // dW_s[V, d_s] = G^T[V, rows] H_s[rows, d_s]: both MN-major, the contraction runs over rows
    e = launch_tc_gemm(G, L.ldG, true, hs_g, ds, true, V, ds, rows_cap, dW, ds, false, nullptr,
                       hdr + 1, nullptr, status, sm_count, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// ---------------------------------------------------------------------------- weight-space audit
// Prefix-versus-full cosine of Section 4.2 in the space of the student's LM-head weight.  The
// candidate lengths L_0 < ... < L_{K-1} (multiples of 64) cut every rollout into K+1 bins of
// positions; dW_bin[i] = G[bin i]^T H_s[bin i] is one GEMM per bin over that bin's 64-row k-blocks,
// the prefix gradient of candidate j is the sum of bins 0..j and the full-horizon reference the sum
// of all bins, so the K cosines come from one pass over the K+1 bin matrices.
constexpr int kMaxCand = 16;
struct CandList {
  int32_t K;
  int32_t L[kMaxCand];
};

namespace {

// k-block lists per bin: entry = first compact gradient row of a 64-row block.
__global__ void lm_bins_kernel(const int32_t* hdr, const int32_t* __restrict__ tiles,
                               const int32_t* __restrict__ g2t, CandList cand, int64_t list_stride,
                               int32_t* lists, int32_t* counts) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  for (int i = 0; i <= cand.K; ++i) counts[i] = 0;
  const int n_gt = hdr[1];
  for (int g = 0; g < n_gt; ++g) {
    const int32_t* e = tiles + (int64_t)g2t[g] * kTileFields;
    for (int h = 0; h < 2; ++h) {
      if (64 * h >= e[3]) continue;          // no gradient row in this half
      const int t = e[1] + 64 * h;
      int bin = 0;
      while (bin < cand.K && cand.L[bin] <= t) ++bin;
      lists[bin * list_stride + counts[bin]++] = g * kBM + 64 * h;
    }
  }
}

// Per block: sums over its share of the elements of  pre_j * full,  pre_j^2  (j < K)  and full^2,
// where pre_j = sum of bins 0..j and full = sum of all bins.  Fixed order inside the block.
constexpr int kGramThreads = 256;
__global__ void __launch_bounds__(kGramThreads) lm_gram_kernel(const float* __restrict__ bins,
                                                               int64_t n_elem, int K,
                                                               double* partial) {
  // fully unrolled over the compile-time bound with run-time guards, so that the accumulators
  // stay in registers
  double acc[2 * kMaxCand + 1];
#pragma unroll
  for (int i = 0; i < 2 * kMaxCand + 1; ++i) acc[i] = 0.0;
  for (int64_t e = (int64_t)blockIdx.x * kGramThreads + threadIdx.x; e < n_elem;
       e += (int64_t)gridDim.x * kGramThreads) {
    float pre[kMaxCand + 1];
    float run = 0.f;
#pragma unroll
    for (int i = 0; i <= kMaxCand; ++i) {
      if (i <= K) run += bins[(int64_t)i * n_elem + e];
      pre[i] = run;
    }
    const double full = (double)run;
#pragma unroll
    for (int j = 0; j < kMaxCand; ++j) {
      if (j < K) {
        acc[2 * j] += (double)pre[j] * full;
        acc[2 * j + 1] += (double)pre[j] * (double)pre[j];
      }
    }
    acc[2 * kMaxCand] += full * full;
  }
  __shared__ double red[kGramThreads];
#pragma unroll
  for (int i = 0; i < 2 * kMaxCand + 1; ++i) {
    if (i >= 2 * K && i != 2 * kMaxCand) continue;     // unused slots (uniform across the block)
    red[threadIdx.x] = acc[i];
    __syncthreads();
    for (int o = kGramThreads / 2; o > 0; o >>= 1) {
      if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
      __syncthreads();
    }
    if (threadIdx.x == 0) partial[(int64_t)blockIdx.x * (2 * kMaxCand + 1) + i] = red[0];
    __syncthreads();
  }
}

// batch_stats[j] = { rho_w(L_j), snr, admissible (0/1), n_tokens }; L_next; flags.
__global__ void lm_align_finish_kernel(const double* __restrict__ partial, int n_blocks,
                                       CandList cand, double rho_star,
                                       const int32_t* __restrict__ rollout_len, int64_t B,
                                       int64_t T, double* batch_stats, int32_t* L_next,
                                       int32_t* flags_out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const int K = cand.K;
  double tot[2 * kMaxCand + 1];
  for (int i = 0; i < 2 * kMaxCand + 1; ++i) {
    double a = 0.0;
    if (i < 2 * K || i == 2 * kMaxCand)
      for (int b = 0; b < n_blocks; ++b) a += partial[(int64_t)b * (2 * kMaxCand + 1) + i];
    tot[i] = a;
  }
  int flags = 0, best = -1;
  const double nf = tot[2 * kMaxCand];
  for (int j = 0; j < K; ++j) {
    double rho;
    if (!(nf > 0.0)) {
      rho = 1.0;
      flags |= ADWIN_ALIGN_DEGENERATE;
    } else {
      rho = tot[2 * j + 1] > 0.0 ? tot[2 * j] / (sqrt(tot[2 * j + 1]) * sqrt(nf)) : 0.0;
    }
    double ntok = 0.0;
    for (int64_t b = 0; b < B; ++b) {
      int64_t R = rollout_len ? rollout_len[b] : T;
      R = R < 0 ? 0 : (R > T ? T : R);
      ntok += (double)(cand.L[j] < R ? cand.L[j] : R);
    }
    const double r2 = rho * rho;
    batch_stats[j * 4 + 0] = rho;
    batch_stats[j * 4 + 1] = r2 < 1.0 ? r2 / (1.0 - r2) : INFINITY;
    batch_stats[j * 4 + 2] = rho >= rho_star ? 1.0 : 0.0;
    batch_stats[j * 4 + 3] = ntok;
    if (rho >= rho_star && best < 0) best = cand.L[j];   // candidates ascend: the first is the shortest
  }
  if (best < 0) {
    best = cand.L[K - 1];
    flags |= ADWIN_ALIGN_NONE_ADMISSIBLE;
  }
  *L_next = best;
  *flags_out = flags;
}

struct AlignLayout {
  size_t off_lists, off_counts, off_bins, off_partial, total;
  int64_t list_stride;
  int gram_blocks;
};

AlignLayout align_layout(const LmLayout& L, int64_t V, int64_t ds, int K) {
  auto up = [](size_t x) { return (x + 1023) & ~size_t(1023); };
  AlignLayout A;
  A.list_stride = 2 * L.max_tiles;
  A.gram_blocks = 1184;
  size_t o = L.total;
  A.off_lists = o;    o = up(o + (size_t)(K + 1) * A.list_stride * 4);
  A.off_counts = o;   o = up(o + (size_t)(K + 1) * 4);
  A.off_bins = o;     o = up(o + (size_t)(K + 1) * (size_t)V * ds * 4);
  A.off_partial = o;  o = up(o + (size_t)A.gram_blocks * (2 * kMaxCand + 1) * 8);
  A.total = o;
  return A;
}

}  // namespace

size_t lmhead_align_workspace_bytes(int64_t B, int64_t T, int64_t V, int64_t ds, int64_t dt,
                                    int64_t max_rows, int K) {
  return align_layout(lm_layout(B, T, V, ds, dt, max_rows, true, false), V, ds, K).total;
}

cudaError_t launch_lmhead_weight_align(const void* hs, const void* ws, const void* ht,
                                       const void* wt, int64_t B, int64_t T, int64_t V, int64_t ds,
                                       int64_t dt, const int32_t* tokens,
                                       const int32_t* rollout_len, const int32_t* cand_host, int K,
                                       double rho_star, int mode, float* kl, float* logratio,
                                       float* gsq, double* batch_stats, int32_t* L_next,
                                       int32_t* flags_out, void* workspace, int64_t max_rows,
                                       int32_t* status, int sm_count, cudaStream_t s) {
  const LmLayout L = lm_layout(B, T, V, ds, dt, max_rows, true, false);
  const AlignLayout A = align_layout(L, V, ds, K);
  char* wb = static_cast<char*>(workspace);
  // every position of every rollout carries gradient here: the window is the rollout itself
  // (window == NULL stands for W_b = T in the row map, so E_b = R_b)
  cudaError_t e = launch_lmhead(hs, ws, ht, wt, B, T, V, ds, dt, tokens, nullptr, rollout_len, 1.0f,
                                mode, 0, nullptr, ADWIN_F32, nullptr, kl, logratio, gsq, nullptr,
                                nullptr, workspace, max_rows, status, sm_count, s, true);
  if (e != cudaSuccess) return e;
  const int32_t* hdr = reinterpret_cast<const int32_t*>(wb + L.off_hdr);
  const int32_t* tiles = reinterpret_cast<const int32_t*>(wb + L.off_tiles);
  const int32_t* g2t = reinterpret_cast<const int32_t*>(wb + L.off_g2t);
  const __nv_bfloat16* hs_c = reinterpret_cast<const __nv_bfloat16*>(wb + L.off_hs);
  const __nv_bfloat16* G = reinterpret_cast<const __nv_bfloat16*>(wb + L.off_G);
  int32_t* lists = reinterpret_cast<int32_t*>(wb + A.off_lists);
  int32_t* counts = reinterpret_cast<int32_t*>(wb + A.off_counts);
  float* bins = reinterpret_cast<float*>(wb + A.off_bins);
  double* partial = reinterpret_cast<double*>(wb + A.off_partial);
  CandList cand;
  cand.K = K;
  for (int i = 0; i < kMaxCand; ++i) cand.L[i] = i < K ? cand_host[i] : 0;
  lm_bins_kernel<<<1, 32, 0, s>>>(hdr, tiles, g2t, cand, A.list_stride, lists, counts);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  const int64_t rows_cap = L.max_tiles * kBM;
  for (int i = 0; i <= K; ++i) {
    e = launch_tc_gemm(G, L.ldG, true, hs_c, ds, true, V, ds, rows_cap,
                       bins + (size_t)i * V * ds, ds, false, nullptr, nullptr, nullptr, status,
                       sm_count, s, lists + (size_t)i * A.list_stride, counts + i);
    if (e != cudaSuccess) return e;
  }
  lm_gram_kernel<<<A.gram_blocks, kGramThreads, 0, s>>>(bins, V * ds, K, partial);
  lm_align_finish_kernel<<<1, 32, 0, s>>>(partial, A.gram_blocks, cand, rho_star, rollout_len, B, T,
                                          batch_stats, L_next, flags_out);
  return cudaGetLastError();
}

}  // namespace adwin
