// Exact full-vocabulary divergence between the rollout policy and the trainer policy, streamed from their two logits
// tensors without materialising a probability tensor: per row TV = 1/2 sum |mu - pi|, KL(mu || pi) and the entropy of pi.
// This is what the Binary / Top-K approximations stand in for (App. B) and what makes the "memory-prohibitive" exact
// quantity available as a monitor.  One CTA walks rows blockIdx.x, +gridDim.x, ...:
//   sweep 1  online sums of both rows: (m, S, A = sum e^(z-m) z) for pi and (m', S', B = sum e^(z'-m') (z' - z)) for mu
//            -> lse, entropy = lse - A/S, KL = B/S' - lse' + lse
//   sweep 2  TV = 1/2 sum |e^(z'-lse') - e^(z-lse)|   (second read of both rows, normally from L2)
#include "dppo_common.cuh"

namespace dppo {
namespace {

constexpr int kThreads = 512;

struct ExactParams {
  const void* z; const void* zmu;
  int64_t T, V, ld_z, ld_mu;
  const uint8_t* token_mask;
  float* tv; float* kl; float* entropy;
  int32_t* status;
};

// running (max, sum e^(x-max), sum e^(x-max) * w): rescaled when the maximum moves
struct Acc3 {
  float m, s, a;
  __device__ __forceinline__ void add(float x, float w) {
    if (!(x <= m)) {                                    // larger, or NaN (which then poisons the sums as it must)
      const float f = ex2_approx((m - x) * kLog2e);     // m = -inf gives 0
      s *= f; a *= f; m = x;
    }
    if (m != -INFINITY) {
      const float e = ex2_approx((x - m) * kLog2e);
      s += e;
      a = fmaf(e, (e > 0.f) ? w : 0.f, a);              // e = 0 (x = -inf): contributes nothing even if w is inf/nan
    }
  }
  __device__ __forceinline__ void merge(const Acc3& o) {
    const float mn = fmaxf(m, o.m);
    if (mn == -INFINITY) return;
    const float f1 = ex2_approx((m - mn) * kLog2e), f2 = ex2_approx((o.m - mn) * kLog2e);
    s = s * f1 + o.s * f2;
    a = a * f1 + o.a * f2;
    m = mn;
  }
};

template <typename InT>
__device__ __forceinline__ void load8(const InT* p, int64_t j, int64_t V, bool vec, float* out, int& n);
template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, int64_t j, int64_t V, bool vec, float* out, int& n) {
  if (vec && j + 8 <= V) {
    const uint4 v = *reinterpret_cast<const uint4*>(p + j);
    out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xffff0000u);
    out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xffff0000u);
    out[4] = __uint_as_float(v.z << 16); out[5] = __uint_as_float(v.z & 0xffff0000u);
    out[6] = __uint_as_float(v.w << 16); out[7] = __uint_as_float(v.w & 0xffff0000u);
    n = 8;
  } else {
    n = 0;
    for (int i = 0; i < 8 && j + i < V; ++i) out[n++] = __bfloat162float(p[j + i]);
  }
}
template <>
__device__ __forceinline__ void load8<float>(const float* p, int64_t j, int64_t V, bool vec, float* out, int& n) {
  if (vec && j + 8 <= V) {
    const float4 a = *reinterpret_cast<const float4*>(p + j), b = *reinterpret_cast<const float4*>(p + j + 4);
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w; out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    n = 8;
  } else {
    n = 0;
    for (int i = 0; i < 8 && j + i < V; ++i) out[n++] = p[j + i];
  }
}

template <typename InT>
__global__ void __launch_bounds__(kThreads) dppo_exact_kernel(ExactParams p, int vec_ok) {
  __shared__ Acc3 s_pi[kThreads / 32], s_mu[kThreads / 32];
  __shared__ double s_tv[kThreads / 32];
  __shared__ float s_lse[2];
  __shared__ int s_bad;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const InT* Z = reinterpret_cast<const InT*>(p.z);
  const InT* ZM = reinterpret_cast<const InT*>(p.zmu);
  for (int64_t t = blockIdx.x; t < p.T; t += gridDim.x) {
    if (p.token_mask && p.token_mask[t] == 0) {
      if (tid == 0) { p.tv[t] = 0.f; p.kl[t] = 0.f; p.entropy[t] = 0.f; }
      continue;
    }
    const InT* z = Z + t * p.ld_z;
    const InT* zm = ZM + t * p.ld_mu;
    // ---- sweep 1
    Acc3 api{-INFINITY, 0.f, 0.f}, amu{-INFINITY, 0.f, 0.f};
    for (int64_t j = (int64_t)tid * 8; j < p.V; j += (int64_t)kThreads * 8) {
      float a[8], b[8];
      int n, n2;
      load8<InT>(z, j, p.V, vec_ok, a, n);
      load8<InT>(zm, j, p.V, vec_ok, b, n2);
      for (int i = 0; i < n; ++i) { api.add(a[i], a[i]); amu.add(b[i], b[i] - a[i]); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Acc3 x{__shfl_xor_sync(0xffffffffu, api.m, o), __shfl_xor_sync(0xffffffffu, api.s, o), __shfl_xor_sync(0xffffffffu, api.a, o)};
      Acc3 y{__shfl_xor_sync(0xffffffffu, amu.m, o), __shfl_xor_sync(0xffffffffu, amu.s, o), __shfl_xor_sync(0xffffffffu, amu.a, o)};
      api.merge(x);
      amu.merge(y);
    }
    if (lane == 0) { s_pi[warp] = api; s_mu[warp] = amu; }
    __syncthreads();
    if (tid == 0) {
      // fixed order, double precision
      float mp = -INFINITY, mq = -INFINITY;
      for (int w = 0; w < kThreads / 32; ++w) { mp = fmaxf(mp, s_pi[w].m); mq = fmaxf(mq, s_mu[w].m); }
      double Sp = 0, Ap = 0, Sq = 0, Bq = 0;
      for (int w = 0; w < kThreads / 32; ++w) {
        if (s_pi[w].s > 0.f || s_pi[w].s != s_pi[w].s) { const double f = exp((double)s_pi[w].m - (double)mp); Sp += f * s_pi[w].s; Ap += f * s_pi[w].a; }
        if (s_mu[w].s > 0.f || s_mu[w].s != s_mu[w].s) { const double f = exp((double)s_mu[w].m - (double)mq); Sq += f * s_mu[w].s; Bq += f * s_mu[w].a; }
      }
      const double lse_p = (double)mp + log(Sp), lse_q = (double)mq + log(Sq);
      const bool ok = isfinite(lse_p) && isfinite(lse_q);
      s_bad = ok ? 0 : 1;
      s_lse[0] = (float)lse_p;
      s_lse[1] = (float)lse_q;
      if (ok) {
        p.entropy[t] = (float)(lse_p - Ap / Sp);
        p.kl[t] = (float)(Bq / Sq - lse_q + lse_p);
      } else {
        p.entropy[t] = 0.f; p.kl[t] = 0.f; p.tv[t] = 0.f;
        atomicOr(p.status, DPPO_STATUS_NONFINITE_ROW);
      }
    }
    __syncthreads();
    if (s_bad) { __syncthreads(); continue; }
    // ---- sweep 2: total variation with both normalisers known
    const float cp = -s_lse[0] * kLog2e, cq = -s_lse[1] * kLog2e;
    float acc = 0.f;
    for (int64_t j = (int64_t)tid * 8; j < p.V; j += (int64_t)kThreads * 8) {
      float a[8], b[8];
      int n, n2;
      load8<InT>(z, j, p.V, vec_ok, a, n);
      load8<InT>(zm, j, p.V, vec_ok, b, n2);
      for (int i = 0; i < n; ++i) acc += fabsf(ex2_approx(fmaf(b[i], kLog2e, cq)) - ex2_approx(fmaf(a[i], kLog2e, cp)));
    }
    double d = (double)acc;
    d = warp_sum(d);
    if (lane == 0) s_tv[warp] = d;
    __syncthreads();
    if (tid == 0) {
      double tot = 0;
      for (int w = 0; w < kThreads / 32; ++w) tot += s_tv[w];
      p.tv[t] = (float)(0.5 * tot);
    }
    __syncthreads();
  }
}

}  // namespace
}  // namespace dppo

extern "C" int dppo_exact_divergence(const void* logits, const void* mu_logits, int64_t T, int64_t V,
                                     int64_t logits_row_stride, int64_t mu_row_stride, int dtype,
                                     const uint8_t* token_mask, float* tv, float* kl, float* entropy,
                                     int32_t* status, void* cuda_stream) {
  using namespace dppo;
  if (T < 0 || V < 1) return DPPO_ERR_SHAPE;
  if (dtype != DPPO_F32 && dtype != DPPO_BF16) return DPPO_ERR_DTYPE;
  if (!status) return DPPO_ERR_NULL;
  if (T > 0 && (!logits || !mu_logits || !tv || !kl || !entropy)) return DPPO_ERR_NULL;
  if (logits_row_stride < V || mu_row_stride < V) return DPPO_ERR_STRIDE;
  const size_t esz = dtype == DPPO_BF16 ? 2 : 4;
  if (((uintptr_t)logits % esz) || ((uintptr_t)mu_logits % esz)) return DPPO_ERR_ALIGN;
  if (T == 0) return DPPO_OK;
  ExactParams p = {logits, mu_logits, T, V, logits_row_stride, mu_row_stride, token_mask, tv, kl, entropy, status};
  const int vec_ok = ((uintptr_t)logits % 16 == 0) && ((uintptr_t)mu_logits % 16 == 0) &&
                     ((logits_row_stride * esz) % 16 == 0) && ((mu_row_stride * esz) % 16 == 0);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t want = (int64_t)sms * 4;
  const int grid = (int)(T < want ? T : want);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (dtype == DPPO_BF16) dppo_exact_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(p, vec_ok);
  else dppo_exact_kernel<float><<<grid, kThreads, 0, st>>>(p, vec_ok);
  return cudaGetLastError() == cudaSuccess ? DPPO_OK : DPPO_ERR_CUDA;
}
