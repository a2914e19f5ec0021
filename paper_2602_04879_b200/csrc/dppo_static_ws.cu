// Entry point for callers that cannot allocate device memory: the per-row scratch of
// dppo_loss_fwd_bwd lives in a fixed array that is part of the loaded library image.
#include <mutex>

#include "../../include/dppo.h"
#include <cuda_runtime.h>

namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kStaticBytes = 256 + 3 * ((size_t)DPPO_STATIC_WS_MAX_ROWS * sizeof(float));

// One copy per GPU that loads the library, held until the process exits.  In host code this name
// is only a handle for the runtime; the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_ws[kStaticBytes];

std::mutex g_mu;
void* g_ws_ptr[kMaxDevices] = {};

// Device address of the array on the current device; looked up once per device and kept for the life of the
// process (so the entry point must not be used again after a cudaDeviceReset of that device: the kept address
// would be stale).
int static_ws_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DPPO_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_ws_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_ws) != cudaSuccess || !ptr) return DPPO_ERR_CUDA;
    g_ws_ptr[dev] = ptr;
  }
  *out = g_ws_ptr[dev];
  return DPPO_OK;
}

}  // namespace

extern "C" int dppo_loss_fwd_bwd_static_ws(const void* logits, int64_t T, int64_t V, int64_t logits_row_stride, int logits_dtype,
                                           const int32_t* sampled_ids, const float* mu_logp,
                                           const int32_t* mu_topk_ids, const float* mu_topk_p,
                                           const float* advantages, const uint8_t* token_mask,
                                           int variant, int K, float delta, const dppo_opts* opts,
                                           float* loss, float* divergence, uint8_t* mask,
                                           void* dlogits, int64_t dlogits_row_stride,
                                           float* stats, int32_t* status, void* cuda_stream) {
  if (T > (int64_t)DPPO_STATIC_WS_MAX_ROWS) return DPPO_ERR_TOO_MANY_ROWS;
  void* ws = nullptr;
  const int rc = static_ws_for_current_device(&ws);
  if (rc != DPPO_OK) return rc;
  // Every call rewrites the header and the per-row entries of its own T rows before it reads them,
  // so nothing in the array has to be cleared between calls.
  return dppo_loss_fwd_bwd(logits, T, V, logits_row_stride, logits_dtype, sampled_ids, mu_logp, mu_topk_ids, mu_topk_p,
                           advantages, token_mask, variant, K, delta, opts, loss, divergence, mask, dlogits,
                           dlogits_row_stride, stats, status, ws, kStaticBytes, cuda_stream);
}
