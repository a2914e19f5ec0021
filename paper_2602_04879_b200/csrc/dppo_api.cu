// C ABI of the DPPO loss library: argument checks, workspace carving, kernel selection, and the
// host-buffer entry point that pipelines copies with the kernels.  See include/dppo.h.
#include <vector>

#include "dppo_common.cuh"
#include "dppo_pipe.cuh"

namespace {

constexpr size_t kAlign = 256;
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t dtype_size(int dt) { return dt == DPPO_BF16 ? 2 : 4; }

}  // namespace

extern "C" {

int dppo_version(void) { return 200; }   // 0.2.0: dppo_opts grew (per-call switches), dppo_workspace_bytes takes the call's shape

size_t dppo_opts_size(void) { return sizeof(dppo_opts); }

const char* dppo_error_string(int code) {
  switch (code) {
    case DPPO_OK: return "ok";
    case DPPO_ERR_NULL: return "a required pointer is NULL";
    case DPPO_ERR_SHAPE: return "bad shape (T < 0, V < 1, K < 0, K > V or d < 1)";
    case DPPO_ERR_DTYPE: return "unknown dtype";
    case DPPO_ERR_VARIANT: return "unknown variant";
    case DPPO_ERR_TOPK: return "Top-K variant with K > 0 needs mu_topk_ids and mu_topk_p";
    case DPPO_ERR_STRIDE: return "row stride smaller than V";
    case DPPO_ERR_ALIGN: return "pointer or stride alignment not usable by the requested kernel";
    case DPPO_ERR_WORKSPACE: return "workspace NULL, misaligned or too small";
    case DPPO_ERR_ALIAS: return "dlogits aliases logits with a different element size or stride";
    case DPPO_ERR_CUDA: return "CUDA runtime error";
    case DPPO_ERR_UNSUPPORTED: return "combination not implemented";
    case DPPO_ERR_TOO_MANY_ROWS: return "T exceeds DPPO_STATIC_WS_MAX_ROWS of the built-in scratch array";
    default: return "unknown error code";
  }
}

size_t dppo_workspace_bytes(int64_t T, int64_t V, int K, int variant) {
  (void)V; (void)K; (void)variant;      // the scratch is per row only: the header and three fp32 columns
  if (T < 0) T = 0;
  return kAlign + 3 * round_up((size_t)T * sizeof(float), kAlign);
}

int dppo_loss_fwd_bwd(const void* logits, int64_t T, int64_t V, int64_t logits_row_stride, int logits_dtype,
                      const int32_t* sampled_ids, const float* mu_logp,
                      const int32_t* mu_topk_ids, const float* mu_topk_p,
                      const float* advantages, const uint8_t* token_mask,
                      int variant, int K, float delta, const dppo_opts* opts,
                      float* loss, float* divergence, uint8_t* mask,
                      void* dlogits, int64_t dlogits_row_stride,
                      float* stats, int32_t* status,
                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
  dppo_opts o = {};
  if (opts) o = *opts;
  if (T < 0 || V < 1 || K < 0 || (int64_t)K > V) return DPPO_ERR_SHAPE;
  if (logits_dtype != DPPO_F32 && logits_dtype != DPPO_BF16) return DPPO_ERR_DTYPE;
  if (o.dlogits_dtype != DPPO_DLOGITS_SAME && o.dlogits_dtype != DPPO_DLOGITS_F32) return DPPO_ERR_DTYPE;
  if (variant < DPPO_BINARY_TV || variant > DPPO_GIVEN_D) return DPPO_ERR_VARIANT;
  if (o.kernel < DPPO_KERNEL_AUTO || o.kernel > DPPO_KERNEL_RING || o.wait_limit_us < 0) return DPPO_ERR_UNSUPPORTED;
  if (o.row_cluster != 0 && o.row_cluster != 1 && o.row_cluster != 2 && o.row_cluster != 4) return DPPO_ERR_UNSUPPORTED;
  if (!loss || !status) return DPPO_ERR_NULL;
  if (T > 0 && (!logits || !sampled_ids || !mu_logp || !advantages || !divergence || !mask || !dlogits)) return DPPO_ERR_NULL;
  const bool topk = (variant == DPPO_TOPK_TV || variant == DPPO_TOPK_KL);
  if (!topk) K = 0;
  if (topk && K > 0 && T > 0 && (!mu_topk_ids || !mu_topk_p)) return DPPO_ERR_TOPK;
  if (logits_row_stride < V || dlogits_row_stride < V) return DPPO_ERR_STRIDE;
  const int out_dtype = (o.dlogits_dtype == DPPO_DLOGITS_F32) ? DPPO_F32 : logits_dtype;
  if (T > 0) {
    // the two tensors are either the same buffer used in place (same element size and row stride) or do not overlap
    // at all: the kernels read rows ahead of the rows they write, so a partial overlap would corrupt rows not yet read
    const uintptr_t in0 = (uintptr_t)logits, in1 = in0 + ((size_t)(T - 1) * logits_row_stride + V) * dtype_size(logits_dtype);
    const uintptr_t out0 = (uintptr_t)dlogits, out1 = out0 + ((size_t)(T - 1) * dlogits_row_stride + V) * dtype_size(out_dtype);
    const bool in_place = (dlogits == logits) && out_dtype == logits_dtype && dlogits_row_stride == logits_row_stride;
    if (!in_place && in0 < out1 && out0 < in1) return DPPO_ERR_ALIAS;
  }
  if (((uintptr_t)logits % dtype_size(logits_dtype)) || ((uintptr_t)dlogits % dtype_size(out_dtype))) return DPPO_ERR_ALIGN;
  if (!workspace || ((uintptr_t)workspace % kAlign) || workspace_bytes < dppo_workspace_bytes(T, V, K, variant)) return DPPO_ERR_WORKSPACE;

  dppo::RowParams p;
  p.logits = logits; p.T = T; p.V = V; p.ld_in = logits_row_stride;
  p.sampled_ids = sampled_ids; p.mu_logp = mu_logp; p.topk_ids = mu_topk_ids; p.topk_p = mu_topk_p;
  p.adv = advantages; p.token_mask = token_mask;
  p.variant = variant; p.K = K; p.delta = delta; p.loss_scale = o.loss_scale; p.is_cap = o.is_cap; p.eps_low = o.eps_low;
  p.wait_ns = dppo::wait_limit_ns(o.wait_limit_us); p.inject = o.test_inject; p.row_cluster = o.row_cluster;
  p.dlogits = dlogits; p.ld_out = dlogits_row_stride;
  p.divergence = divergence; p.mask = mask; p.loss = loss; p.stats = stats; p.status = status;
  char* ws = reinterpret_cast<char*>(workspace);
  const size_t per = round_up((size_t)T * sizeof(float), kAlign);
  p.hdr = reinterpret_cast<dppo::WsHeader*>(ws);
  p.row_loss = reinterpret_cast<float*>(ws + kAlign);
  p.row_r = reinterpret_cast<float*>(ws + kAlign + per);
  p.row_absdiff = reinterpret_cast<float*>(ws + kAlign + 2 * per);

  const bool ring_ok = dppo::ring_layout_ok(p, logits_dtype, out_dtype);
  if (o.kernel == DPPO_KERNEL_RING && !ring_ok) return DPPO_ERR_ALIGN;
  const bool use_ring = (o.kernel == DPPO_KERNEL_RING) || (o.kernel == DPPO_KERNEL_AUTO && ring_ok);

  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (dppo::launch_prelude(p, st) != cudaSuccess) return DPPO_ERR_CUDA;
  cudaError_t e = use_ring ? dppo::launch_ring(p, logits_dtype, out_dtype, st) : dppo::launch_generic(p, logits_dtype, out_dtype, st);
  if (e != cudaSuccess) return DPPO_ERR_CUDA;
  if (dppo::launch_finalize(p, st) != cudaSuccess) return DPPO_ERR_CUDA;
  return DPPO_OK;
}

// ------------------------------------------------------------------------------- host buffers
namespace {
constexpr int kLossSlots = 4096;       // per-chunk losses kept on the device between two reads by the host
struct StageLayout {
  size_t logits, dlogits, ids, mu_logp, adv, tmask, topk_ids, topk_p, D, M, ws, total;
  bool in_place;
};
StageLayout stage_layout(int64_t R, int64_t V, int K, int in_dt, int out_dt) {
  StageLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += round_up(bytes ? bytes : 1, kAlign); return o; };
  L.in_place = (in_dt == out_dt);
  L.logits = take((size_t)R * V * dtype_size(in_dt));
  L.dlogits = L.in_place ? L.logits : take((size_t)R * V * dtype_size(out_dt));
  L.ids = take((size_t)R * 4);
  L.mu_logp = take((size_t)R * 4);
  L.adv = take((size_t)R * 4);
  L.tmask = take((size_t)R);
  L.topk_ids = take((size_t)R * K * 4);
  L.topk_p = take((size_t)R * K * 4);
  L.D = take((size_t)R * 4);
  L.M = take((size_t)R);
  L.ws = take(dppo_workspace_bytes(R, V, K, 0));
  L.total = off;
  return L;
}
}  // namespace

size_t dppo_host_staging_bytes(int64_t rows_per_chunk, int64_t V, int K, int logits_dtype, int dlogits_dtype) {
  if (rows_per_chunk < 1 || V < 1 || K < 0) return 0;
  const int out_dt = (dlogits_dtype == DPPO_DLOGITS_F32) ? DPPO_F32 : logits_dtype;
  return 2 * stage_layout(rows_per_chunk, V, K, logits_dtype, out_dt).total + round_up(kLossSlots * sizeof(float), kAlign) + kAlign;
}

int dppo_loss_fwd_bwd_host(const void* logits, int64_t T, int64_t V, int logits_dtype,
                           const int32_t* sampled_ids, const float* mu_logp,
                           const int32_t* mu_topk_ids, const float* mu_topk_p,
                           const float* advantages, const uint8_t* token_mask,
                           int variant, int K, float delta, const dppo_opts* opts,
                           float* loss_host, float* divergence_host, uint8_t* mask_host,
                           void* dlogits_host, int32_t* status_host,
                           void* staging, size_t staging_bytes, int64_t rows_per_chunk) {
  dppo_opts o = {};
  if (opts) o = *opts;
  if (T < 0 || V < 1 || K < 0 || (int64_t)K > V || rows_per_chunk < 1) return DPPO_ERR_SHAPE;
  if (logits_dtype != DPPO_F32 && logits_dtype != DPPO_BF16) return DPPO_ERR_DTYPE;
  if (o.dlogits_dtype != DPPO_DLOGITS_SAME && o.dlogits_dtype != DPPO_DLOGITS_F32) return DPPO_ERR_DTYPE;
  if (variant < DPPO_BINARY_TV || variant > DPPO_MINIMAL_MASK) return DPPO_ERR_VARIANT;
  if (!loss_host || !status_host) return DPPO_ERR_NULL;
  if (T > 0 && (!logits || !sampled_ids || !mu_logp || !advantages || !divergence_host || !mask_host)) return DPPO_ERR_NULL;
  const bool topk = (variant == DPPO_TOPK_TV || variant == DPPO_TOPK_KL);
  if (!topk) K = 0;
  if (topk && K > 0 && T > 0 && (!mu_topk_ids || !mu_topk_p)) return DPPO_ERR_TOPK;
  const int out_dt = (o.dlogits_dtype == DPPO_DLOGITS_F32) ? DPPO_F32 : logits_dtype;
  const int64_t R = rows_per_chunk;
  const int64_t nchunks = (T + R - 1) / R;
  if (!staging || ((uintptr_t)staging % kAlign) || staging_bytes < dppo_host_staging_bytes(R, V, K, logits_dtype, o.dlogits_dtype))
    return DPPO_ERR_WORKSPACE;

  // token-mean scale over the whole batch, counted on the host
  int64_t n_valid = T;
  if (token_mask) { n_valid = 0; for (int64_t t = 0; t < T; ++t) n_valid += (token_mask[t] != 0); }
  dppo_opts oc = o;
  oc.loss_scale = (o.loss_scale > 0.f) ? o.loss_scale : (n_valid > 0 ? (float)(1.0 / (double)n_valid) : 1.0f);

  *loss_host = 0.f;
  *status_host = 0;
  if (T == 0) return DPPO_OK;

  const StageLayout L = stage_layout(R, V, K, logits_dtype, out_dt);
  char* base = reinterpret_cast<char*>(staging);
  float* d_loss_parts = reinterpret_cast<float*>(base + 2 * L.total);
  // one status word for all chunks: the kernels only ever OR bits into it
  int32_t* d_status = reinterpret_cast<int32_t*>(base + 2 * L.total + round_up(kLossSlots * sizeof(float), kAlign));
  cudaStream_t st[2] = {nullptr, nullptr};
  cudaEvent_t zeroed = nullptr;
  int rc = DPPO_OK;
  if (cudaStreamCreateWithFlags(&st[0], cudaStreamNonBlocking) != cudaSuccess) return DPPO_ERR_CUDA;
  if (cudaStreamCreateWithFlags(&st[1], cudaStreamNonBlocking) != cudaSuccess) { cudaStreamDestroy(st[0]); return DPPO_ERR_CUDA; }
  if (cudaEventCreateWithFlags(&zeroed, cudaEventDisableTiming) != cudaSuccess) { cudaStreamDestroy(st[0]); cudaStreamDestroy(st[1]); return DPPO_ERR_CUDA; }
  const size_t isz = dtype_size(logits_dtype), osz = dtype_size(out_dt);
  std::vector<float> loss_parts((size_t)(nchunks < kLossSlots ? nchunks : kLossSlots), 0.f);
  double loss_acc = 0.0;
  int64_t parts_pending = 0;        // chunk losses on the device that the host has not added yet
#define DPPO_TRY(call) do { if ((call) != cudaSuccess) { rc = DPPO_ERR_CUDA; goto done; } } while (0)
  DPPO_TRY(cudaMemsetAsync(d_status, 0, 4, st[0]));
  DPPO_TRY(cudaEventRecord(zeroed, st[0]));
  DPPO_TRY(cudaStreamWaitEvent(st[1], zeroed, 0));
  for (int64_t c = 0; c < nchunks; ++c) {
    const int b = (int)(c & 1);
    cudaStream_t s = st[b];
    char* sb = base + (size_t)b * L.total;
    const int64_t r0 = c * R, n = (T - r0 < R) ? (T - r0) : R;
    if (parts_pending == kLossSlots) {       // every slot holds a chunk's loss: collect them before they are reused
      DPPO_TRY(cudaStreamSynchronize(st[0]));
      DPPO_TRY(cudaStreamSynchronize(st[1]));
      DPPO_TRY(cudaMemcpy(loss_parts.data(), d_loss_parts, (size_t)parts_pending * sizeof(float), cudaMemcpyDeviceToHost));
      for (int64_t i = 0; i < parts_pending; ++i) loss_acc += (double)loss_parts[(size_t)i];
      parts_pending = 0;
    }
    DPPO_TRY(cudaMemcpyAsync(sb + L.logits, (const char*)logits + (size_t)r0 * V * isz, (size_t)n * V * isz, cudaMemcpyHostToDevice, s));
    DPPO_TRY(cudaMemcpyAsync(sb + L.ids, sampled_ids + r0, (size_t)n * 4, cudaMemcpyHostToDevice, s));
    DPPO_TRY(cudaMemcpyAsync(sb + L.mu_logp, mu_logp + r0, (size_t)n * 4, cudaMemcpyHostToDevice, s));
    DPPO_TRY(cudaMemcpyAsync(sb + L.adv, advantages + r0, (size_t)n * 4, cudaMemcpyHostToDevice, s));
    if (token_mask) DPPO_TRY(cudaMemcpyAsync(sb + L.tmask, token_mask + r0, (size_t)n, cudaMemcpyHostToDevice, s));
    if (K > 0) {
      DPPO_TRY(cudaMemcpyAsync(sb + L.topk_ids, mu_topk_ids + (size_t)r0 * K, (size_t)n * K * 4, cudaMemcpyHostToDevice, s));
      DPPO_TRY(cudaMemcpyAsync(sb + L.topk_p, mu_topk_p + (size_t)r0 * K, (size_t)n * K * 4, cudaMemcpyHostToDevice, s));
    }
    {
      int e = dppo_loss_fwd_bwd(sb + L.logits, n, V, V, logits_dtype,
                                (const int32_t*)(sb + L.ids), (const float*)(sb + L.mu_logp),
                                K > 0 ? (const int32_t*)(sb + L.topk_ids) : nullptr, K > 0 ? (const float*)(sb + L.topk_p) : nullptr,
                                (const float*)(sb + L.adv), token_mask ? (const uint8_t*)(sb + L.tmask) : nullptr,
                                variant, K, delta, &oc, d_loss_parts + parts_pending, (float*)(sb + L.D), (uint8_t*)(sb + L.M),
                                sb + L.dlogits, V, nullptr, d_status, sb + L.ws, dppo_workspace_bytes(R, V, K, variant), s);
      if (e != DPPO_OK) { rc = e; goto done; }
      ++parts_pending;
    }
    DPPO_TRY(cudaMemcpyAsync(divergence_host + r0, sb + L.D, (size_t)n * 4, cudaMemcpyDeviceToHost, s));
    DPPO_TRY(cudaMemcpyAsync(mask_host + r0, sb + L.M, (size_t)n, cudaMemcpyDeviceToHost, s));
    if (dlogits_host)
      DPPO_TRY(cudaMemcpyAsync((char*)dlogits_host + (size_t)r0 * V * osz, sb + L.dlogits, (size_t)n * V * osz, cudaMemcpyDeviceToHost, s));
  }
  DPPO_TRY(cudaStreamSynchronize(st[0]));
  DPPO_TRY(cudaStreamSynchronize(st[1]));
  DPPO_TRY(cudaMemcpy(loss_parts.data(), d_loss_parts, (size_t)parts_pending * sizeof(float), cudaMemcpyDeviceToHost));
  for (int64_t i = 0; i < parts_pending; ++i) loss_acc += (double)loss_parts[(size_t)i];
  {
    int32_t stt = 0;
    DPPO_TRY(cudaMemcpy(&stt, d_status, 4, cudaMemcpyDeviceToHost));
    *loss_host = (float)loss_acc;
    *status_host = stt;
  }
done:
#undef DPPO_TRY
  cudaStreamSynchronize(st[0]);
  cudaStreamSynchronize(st[1]);
  cudaEventDestroy(zeroed);
  cudaStreamDestroy(st[0]);
  cudaStreamDestroy(st[1]);
  return rc;
}

}  // extern "C"
