// adwin_opd_kl_fwd_bwd_no_alloc: the windowed divergence pass for callers that have no device
// memory to hand over as a workspace and are not in a position to allocate any.
//
// The row map (effective windows and their prefix sums) that the kernels read is the only
// scratch the pass needs.  Here it lives in a file-scope array in device memory that is part of
// the library image: every GPU that loads the library carries these 66 KB until the process
// exits, and nothing is allocated or freed at any time.
#include <mutex>

#include "adwin_internal.h"

namespace adwin {
namespace {

// Large enough for the row map of kNoAllocMaxSequences sequences:
// 256 (header) + 8*(B+1) rounded up to 256 + 2 * 4*B  =  256 + 33024 + 16384 + 16384.
constexpr int64_t kNoAllocMaxSequences = 4096;
constexpr size_t kScratchBytes = 66048;

static __device__ __align__(256) unsigned char g_rowmap_scratch[kScratchBytes];

// In host code `g_rowmap_scratch` is only a handle for the runtime, not an address the GPU can
// use, so the device address is looked up once per device (with that device current) and kept.
void* scratch_for_current_device() {
  static std::mutex mu;
  static void* table[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (table[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_rowmap_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return nullptr;
    }
    table[dev] = ptr;
  }
  return table[dev];
}

}  // namespace
}  // namespace adwin

using namespace adwin;

extern "C" {

int64_t adwin_no_alloc_max_sequences(void) { return kNoAllocMaxSequences; }

int adwin_opd_kl_fwd_bwd_no_alloc(const void* student_logits, const void* teacher_logits,
                                  int dtype, int64_t B, int64_t T, int64_t V, int64_t ld,
                                  const int32_t* tokens, const int32_t* window,
                                  const int32_t* rollout_len, float grad_scale, int grad_mode,
                                  int flags, void* grad_student, int grad_dtype, int64_t ld_grad,
                                  float* kl, float* logratio, float* gsq, float* lse_student,
                                  float* lse_teacher, int32_t* dev_status, void* cuda_stream) {
  if (B > kNoAllocMaxSequences) return ADWIN_ERR_WORKSPACE;   // the built-in row map is too small
  if (B > 0 && workspace_layout(B).total > kScratchBytes) return ADWIN_ERR_WORKSPACE;
  void* scratch = scratch_for_current_device();
  if (scratch == nullptr) return ADWIN_ERR_CUDA;
  // Nothing in the array has to start at zero: the row-map kernel of every call rewrites all the
  // entries that the call's other kernels read before they read them (the 256-byte header is
  // reserved and neither read nor written), so nothing a previous call left behind is ever used.
  // Nothing is enqueued here either: the ordinary entry point validates the arguments first.
  return adwin_opd_kl_fwd_bwd(student_logits, teacher_logits, dtype, B, T, V, ld, tokens, window,
                              rollout_len, grad_scale, grad_mode, flags, grad_student, grad_dtype,
                              ld_grad, kl, logratio, gsq, lse_student, lse_teacher, scratch,
                              kScratchBytes, dev_status, cuda_stream);
}

}  // extern "C"
