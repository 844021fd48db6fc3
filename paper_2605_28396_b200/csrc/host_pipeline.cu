// Host-buffer entry point: the same windowed divergence pass for logits that live in host
// memory.  Only rows inside the processed range ever cross PCIe (rows past the window cost no
// transfer either); the copies of stage k+1 and the read-back of stage k-1 overlap the kernels of
// stage k on three streams.  The staging memory on the device belongs to the caller.
#include <cstring>
#include <mutex>

#include "adwin_common.cuh"
#include "adwin_internal.h"

namespace adwin {
namespace {

constexpr int kStages = 3;

struct Pipeline {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t in_ready[kStages], comp_done[kStages], out_done[kStages], start = nullptr;
};

Pipeline* pipeline_for_current_device() {
  static std::mutex mu;
  static Pipeline table[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  Pipeline& p = table[dev];
  if (!p.ready) {
    if (cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    for (int i = 0; i < kStages; ++i) {
      if (cudaEventCreateWithFlags(&p.in_ready[i], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&p.comp_done[i], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&p.out_done[i], cudaEventDisableTiming) != cudaSuccess)
        return nullptr;
    }
    if (cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    p.ready = true;
  }
  return &p;
}

inline size_t up256(size_t x) { return (x + 255) & ~size_t(255); }
inline size_t esize(int dtype) { return dtype == ADWIN_F32 ? 4 : 2; }

struct StageLayout {
  int64_t pitch_in, pitch_out;  // elements
  size_t off_z, off_u, off_tok, off_win, off_rl, off_ws, off_grad, off_kl, off_c, off_q, total;
};

StageLayout stage_layout(int64_t rows, int64_t V, int dtype, int grad_dtype, bool has_grad) {
  StageLayout L;
  const size_t es = esize(dtype), gs = esize(grad_dtype);
  L.pitch_in = (int64_t)((V * es + 15) / 16 * 16 / es);
  L.pitch_out = (int64_t)((V * gs + 15) / 16 * 16 / gs);
  size_t o = 0;
  L.off_z = o;   o = up256(o + (size_t)rows * L.pitch_in * es);
  L.off_u = o;   o = up256(o + (size_t)rows * L.pitch_in * es);
  L.off_tok = o; o = up256(o + (size_t)rows * 4);
  L.off_win = o; o = up256(o + 4);
  L.off_rl = o;  o = up256(o + 4);
  L.off_ws = o;  o = up256(o + workspace_layout(1).total);
  L.off_grad = o; o = up256(o + (has_grad ? (size_t)rows * L.pitch_out * gs : 0));
  L.off_kl = o;  o = up256(o + (size_t)rows * 4);
  L.off_c = o;   o = up256(o + (size_t)rows * 4);
  L.off_q = o;   o = up256(o + (size_t)rows * 4);
  L.total = o;
  return L;
}

__global__ void set_lengths_kernel(int32_t* win, int32_t* rl, int32_t w, int32_t r) {
  *win = w;
  *rl = r;
}

}  // namespace
}  // namespace adwin

using namespace adwin;

extern "C" {

size_t adwin_host_staging_bytes(int64_t rows_per_stage, int64_t V, int dtype, int grad_dtype,
                                int with_grad) {
  if (rows_per_stage < 1 || V < 1) return 0;
  return kStages * stage_layout(rows_per_stage, V, dtype, grad_dtype, with_grad != 0).total;
}

int adwin_opd_kl_fwd_bwd_host(const void* student_host, const void* teacher_host, int dtype,
                              int64_t B, int64_t T, int64_t V, int64_t ld,
                              const int32_t* tokens_host, const int32_t* window_host,
                              const int32_t* rollout_len_host, float grad_scale, int grad_mode,
                              int flags, void* grad_host, int grad_dtype, int64_t ld_grad,
                              float* kl_host, float* logratio_host, float* gsq_host,
                              void* staging_dev, size_t staging_bytes, int64_t rows_per_stage,
                              int32_t* dev_status, void* cuda_stream) {
  if (dtype != ADWIN_F32 && dtype != ADWIN_BF16) return ADWIN_ERR_DTYPE;
  if (grad_host && grad_dtype != ADWIN_F32 && grad_dtype != ADWIN_BF16) return ADWIN_ERR_DTYPE;
  if (B < 0 || T < 0 || V < 1 || ld < V || rows_per_stage < 1) return ADWIN_ERR_SHAPE;
  if (grad_host && ld_grad < V) return ADWIN_ERR_SHAPE;
  if (!dev_status) return ADWIN_ERR_NULL;
  if (B == 0 || T == 0) return ADWIN_OK;
  if (!student_host || !teacher_host || !tokens_host || !window_host || !kl_host || !logratio_host)
    return ADWIN_ERR_NULL;
  const bool has_grad = grad_host != nullptr;
  const int gd = has_grad ? grad_dtype : dtype;
  const StageLayout L = stage_layout(rows_per_stage, V, dtype, gd, has_grad);
  if (!staging_dev || (reinterpret_cast<uintptr_t>(staging_dev) & 255) ||
      staging_bytes < kStages * L.total)
    return ADWIN_ERR_WORKSPACE;
  for (int64_t b = 0; b < B; ++b) {
    const int64_t r = rollout_len_host ? rollout_len_host[b] : T;
    if (window_host[b] < 0 || r < 0 || r > T) return ADWIN_ERR_WINDOW;
  }
  Pipeline* pl = pipeline_for_current_device();
  if (!pl) return ADWIN_ERR_CUDA;
  cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
  const size_t es = esize(dtype), gs = esize(gd);

  // Rows that are not processed report 0; tail gradient rows are zeroed on request.
  std::memset(kl_host, 0, (size_t)B * T * 4);
  std::memset(logratio_host, 0, (size_t)B * T * 4);
  if (gsq_host) std::memset(gsq_host, 0, (size_t)B * T * 4);

  // The copy streams start after whatever the caller already enqueued.
  if (cudaEventRecord(pl->start, user) != cudaSuccess) return ADWIN_ERR_CUDA;
  cudaStreamWaitEvent(pl->in, pl->start, 0);
  cudaStreamWaitEvent(pl->out, pl->start, 0);

  int64_t k = 0;  // stage counter
  for (int64_t b = 0; b < B; ++b) {
    const int64_t R = rollout_len_host ? rollout_len_host[b] : T;
    const int64_t E = window_host[b] < R ? window_host[b] : R;
    const int64_t P = (flags & ADWIN_RANGE_FULL) ? R : E;
    if (has_grad && (flags & ADWIN_ZERO_TAIL)) {
      for (int64_t t = E; t < T; ++t)
        std::memset(static_cast<char*>(grad_host) + ((size_t)(b * T + t) * ld_grad) * gs, 0,
                    (size_t)V * gs);
    }
    for (int64_t t0 = 0; t0 < P; t0 += rows_per_stage, ++k) {
      const int64_t rows = (P - t0 < rows_per_stage) ? P - t0 : rows_per_stage;
      const int64_t wrows = E - t0 < 0 ? 0 : (E - t0 < rows ? E - t0 : rows);  // rows with a gradient
      const int s = (int)(k % kStages);
      char* base = static_cast<char*>(staging_dev) + (size_t)s * L.total;
      const size_t row0 = (size_t)(b * T + t0);

      // inputs: reuse of this buffer waits for the kernels that read it
      if (k >= kStages) cudaStreamWaitEvent(pl->in, pl->comp_done[s], 0);
      cudaMemcpy2DAsync(base + L.off_z, L.pitch_in * es,
                        static_cast<const char*>(student_host) + row0 * ld * es, ld * es, V * es,
                        rows, cudaMemcpyHostToDevice, pl->in);
      cudaMemcpy2DAsync(base + L.off_u, L.pitch_in * es,
                        static_cast<const char*>(teacher_host) + row0 * ld * es, ld * es, V * es,
                        rows, cudaMemcpyHostToDevice, pl->in);
      cudaMemcpyAsync(base + L.off_tok, tokens_host + row0, rows * 4, cudaMemcpyHostToDevice,
                      pl->in);
      cudaEventRecord(pl->in_ready[s], pl->in);

      // compute on the caller's stream
      cudaStreamWaitEvent(user, pl->in_ready[s], 0);
      if (k >= kStages) cudaStreamWaitEvent(user, pl->out_done[s], 0);
      set_lengths_kernel<<<1, 1, 0, user>>>(reinterpret_cast<int32_t*>(base + L.off_win),
                                            reinterpret_cast<int32_t*>(base + L.off_rl),
                                            (int32_t)wrows, (int32_t)rows);
      const int rc = adwin_opd_kl_fwd_bwd(
          base + L.off_z, base + L.off_u, dtype, 1, rows, V, L.pitch_in,
          reinterpret_cast<const int32_t*>(base + L.off_tok),
          reinterpret_cast<const int32_t*>(base + L.off_win),
          reinterpret_cast<const int32_t*>(base + L.off_rl), grad_scale, grad_mode,
          flags & ~ADWIN_ZERO_TAIL, has_grad ? base + L.off_grad : nullptr, gd, L.pitch_out,
          reinterpret_cast<float*>(base + L.off_kl), reinterpret_cast<float*>(base + L.off_c),
          reinterpret_cast<float*>(base + L.off_q), nullptr, nullptr, base + L.off_ws,
          workspace_layout(1).total, dev_status, user);
      if (rc != ADWIN_OK) return rc;
      cudaEventRecord(pl->comp_done[s], user);

      // outputs
      cudaStreamWaitEvent(pl->out, pl->comp_done[s], 0);
      if (has_grad && wrows > 0)
        cudaMemcpy2DAsync(static_cast<char*>(grad_host) + row0 * ld_grad * gs, ld_grad * gs,
                          base + L.off_grad, L.pitch_out * gs, V * gs, wrows,
                          cudaMemcpyDeviceToHost, pl->out);
      cudaMemcpyAsync(kl_host + row0, base + L.off_kl, rows * 4, cudaMemcpyDeviceToHost, pl->out);
      cudaMemcpyAsync(logratio_host + row0, base + L.off_c, rows * 4, cudaMemcpyDeviceToHost,
                      pl->out);
      if (gsq_host)
        cudaMemcpyAsync(gsq_host + row0, base + L.off_q, rows * 4, cudaMemcpyDeviceToHost, pl->out);
      cudaEventRecord(pl->out_done[s], pl->out);
    }
  }
  // Completion of the caller's stream implies completion of every read-back.
  const int64_t last = k < kStages ? k : kStages;
  for (int64_t i = 0; i < last; ++i) cudaStreamWaitEvent(user, pl->out_done[i], 0);
  return cudaGetLastError() == cudaSuccess ? ADWIN_OK : ADWIN_ERR_CUDA;
}

}  // extern "C"
