// Prelude / finalize kernels of every call, and the scalar-access row kernel that accepts any
// layout (odd V, unaligned rows).  The fast path for 16-byte aligned layouts is in dppo_ring.cu.
#include "dppo_common.cuh"

namespace dppo {

// ---------------------------------------------------------------------------------------------
// Prelude: N_valid and the scale s of this call.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) dppo_prelude_kernel(RowParams p) {
  __shared__ int s_count;
  if (threadIdx.x == 0) s_count = 0;
  __syncthreads();
  int c = 0;
  if (p.token_mask) {
    for (int64_t t = threadIdx.x; t < p.T; t += blockDim.x) c += (p.token_mask[t] != 0);
  } else {
    for (int64_t t = threadIdx.x; t < p.T; t += blockDim.x) c += 1;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0) atomicAdd(&s_count, c);     // integer: order does not matter
  __syncthreads();
  if (threadIdx.x == 0) {
    p.hdr->n_valid = s_count;
    p.hdr->scale = (p.loss_scale > 0.f) ? (double)p.loss_scale : (s_count > 0 ? 1.0 / (double)s_count : 0.0);
  }
}

// ---------------------------------------------------------------------------------------------
// Finalize: loss = sum_t row_loss[t] in double, fixed order; optional statistics.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) dppo_finalize_kernel(RowParams p, int block_first, int block_last) {
  constexpr int NT = 1024;
  __shared__ double red[6][NT / 32];
  __shared__ float redmax[NT / 32];
  double loss = 0.0, sumD = 0.0, sumAbs = 0.0, sumR = 0.0, sumL = 0.0, nblk = 0.0;
  float maxD = 0.f;
  for (int64_t t = threadIdx.x; t < p.T; t += NT) {
    if (p.token_mask && p.token_mask[t] == 0) continue;
    loss += (double)p.row_loss[t];
    if (p.stats) {
      float D = p.divergence[t];
      if (isfinite(D)) { sumD += (double)D; }
      maxD = fmaxf(maxD, D);
      sumAbs += (double)p.row_absdiff[t];
      sumR += (double)p.row_r[t];
      sumL += fabs((double)p.row_loss[t]);
      // blocked rows among rows that produced outputs (rows dropped for a status bit have r = 0)
      nblk += (p.mask[t] == 0 && p.row_r[t] != 0.f) ? 1.0 : 0.0;
    }
  }
  double v[6] = {loss, sumD, sumAbs, sumR, sumL, nblk};
#pragma unroll
  for (int i = 0; i < 6; ++i) v[i] = warp_sum(v[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) maxD = fmaxf(maxD, __shfl_xor_sync(0xffffffffu, maxD, o));
  int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < 6; ++i) red[i][w] = v[i];
    redmax[w] = maxD;
  }
  __syncthreads();
  if (w == 0) {
#pragma unroll
    for (int i = 0; i < 6; ++i) v[i] = warp_sum(red[i][lane]);
    maxD = redmax[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) maxD = fmaxf(maxD, __shfl_xor_sync(0xffffffffu, maxD, o));
    if (lane == 0) {
      if (!block_first) {          // rows finished by earlier blocks of this call (same stream: a fixed order)
#pragma unroll
        for (int i = 0; i < 6; ++i) v[i] += p.hdr->acc[i];
        maxD = fmaxf(maxD, p.hdr->max_d);
      }
      if (!block_last) {
#pragma unroll
        for (int i = 0; i < 6; ++i) p.hdr->acc[i] = v[i];
        p.hdr->max_d = maxD;
      } else {
        *p.loss = (float)v[0];
        if (p.stats) {
          p.stats[0] = (float)p.hdr->n_valid;
          p.stats[1] = (float)v[5];
          p.stats[2] = (float)v[1];
          p.stats[3] = maxD;
          p.stats[4] = (float)v[2];
          p.stats[5] = (float)v[3];
          p.stats[6] = (float)v[4];
          p.stats[7] = 0.f;
        }
      }
    }
  }
}

cudaError_t launch_prelude(const RowParams& p, cudaStream_t st) {
  dppo_prelude_kernel<<<1, 1024, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_finalize(const RowParams& p, cudaStream_t st, bool block_first, bool block_last) {
  dppo_finalize_kernel<<<1, 1024, 0, st>>>(p, block_first ? 1 : 0, block_last ? 1 : 0);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Scalar-access row kernel: one CTA walks rows blockIdx.x, +gridDim.x, ...; two sweeps per row
// (online log-sum-exp, then the gradient), element-wise loads so that any V / stride works.
// ---------------------------------------------------------------------------------------------
constexpr int kGenericThreads = 512;

template <typename InT, typename OutT>
__global__ void __launch_bounds__(kGenericThreads) dppo_row_generic_kernel(RowParams p) {
  __shared__ float s_m[kGenericThreads / 32], s_s[kGenericThreads / 32];
  __shared__ RowCoef s_coef;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double scale = p.hdr->scale;
  const InT* logits = reinterpret_cast<const InT*>(p.logits);
  OutT* dlogits = reinterpret_cast<OutT*>(p.dlogits);

  for (int64_t t = blockIdx.x; t < p.T; t += gridDim.x) {
    OutT* drow = dlogits + t * p.ld_out;
    const InT* zrow = logits + t * p.ld_in;
    bool valid = p.token_mask ? (p.token_mask[t] != 0) : true;
    int a = 0;
    int flags = 0;
    if (valid) {
      a = p.sampled_ids[t];
      if (a < 0 || (int64_t)a >= p.V) { valid = false; flags |= DPPO_STATUS_BAD_SAMPLED_ID; }
    }
    if (valid) {
      // sweep 1: per-thread online (max, sum of exp) over the entries other than the sampled token's
      float m = -INFINITY, s = 0.f;
      for (int64_t j = tid; j < p.V; j += kGenericThreads) {
        if (j == (int64_t)a) continue;
        float z = to_f32<InT>(zrow[j]);
        if (z > m) {                                  // z is finite or +inf here
          s = s * ex2_approx((m - z) * kLog2e);
          m = z;
        }
        float ref = (m == -INFINITY) ? 0.f : m;
        s += ex2_approx((z - ref) * kLog2e);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
        merge_ms(m, s, m2, s2);
      }
      if (lane == 0) { s_m[warp] = m; s_s[warp] = s; }
    }
    __syncthreads();
    if (warp == 0) {
      RowCoef coef;
      coef.c2 = 0.f; coef.sgn = 0.f; coef.fix = 0.f; coef.zero_row = 1;
      float D = 0.f, r = 0.f, absdiff = 0.f;
      int M = 0;
      double g = 0.0;
      if (valid) {
        // combine the warps' partials in a fixed order, in double
        float mm = -INFINITY;
        for (int w = 0; w < kGenericThreads / 32; ++w) mm = fmaxf(mm, s_m[w]);
        double S = 0.0;
        for (int w = 0; w < kGenericThreads / 32; ++w)
          if (s_s[w] > 0.f || s_s[w] != s_s[w]) S += (double)s_s[w] * exp((double)s_m[w] - (double)mm);
        double lse, log_other;
        combine_lse((double)mm, S, (double)to_f32<InT>(zrow[a]), lse, log_other);
        if (!isfinite(lse)) {
          flags |= DPPO_STATUS_NONFINITE_ROW;
        } else {
          double pi_a;
          int f2 = 0;
          auto z_at = [&](int id, int) { return to_f32<InT>(zrow[id]); };
          row_scalars_warp(p, t, a, lse, log_other, scale, z_at, D, M, g, r, absdiff, pi_a, f2);
          if (f2) { flags |= f2; D = 0.f; M = 0; g = 0.0; r = 0.f; absdiff = 0.f; }
          else coef = make_coef(g, lse, pi_a);
        }
      }
      if (lane == 0) {
        s_coef = coef;
        p.divergence[t] = D;
        p.mask[t] = (uint8_t)M;
        p.row_loss[t] = (float)(-g);
        p.row_r[t] = r;
        p.row_absdiff[t] = absdiff;
        if (flags) atomicOr(p.status, flags);
      }
    }
    __syncthreads();
    const RowCoef coef = s_coef;
    // sweep 2: gradient row
    if (coef.zero_row) {
      for (int64_t j = tid; j < p.V; j += kGenericThreads) drow[j] = from_f32<OutT>(0.f);
    } else {
      for (int64_t j = tid; j < p.V; j += kGenericThreads) {
        float z = to_f32<InT>(zrow[j]);
        float v = coef.sgn * ex2_approx(fmaf(z, kLog2e, coef.c2));
        if (j == (int64_t)a) v = coef.fix;
        drow[j] = from_f32<OutT>(v);
      }
    }
    __syncthreads();   // s_coef / s_m are reused by the next row
  }
}

cudaError_t launch_generic(const RowParams& p, int in_dtype, int out_dtype, cudaStream_t st) {
  if (p.T == 0) return cudaSuccess;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t want = (int64_t)sms * 4;
  int grid = (int)(p.T < want ? p.T : want);
  if (in_dtype == DPPO_F32 && out_dtype == DPPO_F32)
    dppo_row_generic_kernel<float, float><<<grid, kGenericThreads, 0, st>>>(p);
  else if (in_dtype == DPPO_BF16 && out_dtype == DPPO_BF16)
    dppo_row_generic_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, kGenericThreads, 0, st>>>(p);
  else if (in_dtype == DPPO_BF16 && out_dtype == DPPO_F32)
    dppo_row_generic_kernel<__nv_bfloat16, float><<<grid, kGenericThreads, 0, st>>>(p);
  else
    return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace dppo
