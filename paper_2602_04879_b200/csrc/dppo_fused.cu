// Fused LM-head variant of the DPPO loss: logits = hidden x W are produced tile by tile on the tensor cores and
// consumed in the accumulators' epilogue, so the [T, V] logits never exist in memory, and every tile is computed once.
//
// The gradient row is g (softmax(z) - onehot) = (g / S) (E - S onehot) with E_j = exp(z_j - c) and S = sum_j E_j for ANY
// per-row reference c.  With c known before the GEMM (the logit of the sampled token, one dot product per row) the
// exponentials can be written in the same pass that sums them; the per-row factor g / S, known only after the whole
// vocabulary has been seen, is applied later where it is cheap: to the rows of dHidden in that GEMM's epilogue, and to
// the rows of hidden before the dW GEMM.  bf16 has the exponent range of fp32, so E needs no row maximum.
//
//   1. partition      valid rows with a non-zero advantage first, then the other valid rows (they need the divergence
//                     but no gradient), packed copies of hidden / sampled ids; (Top-K variants) W^T for the gather
//   2. reference      c_t = z_t[a_t] by a dot product per row
//   3. forward GEMM   z-tile = hidden . W-tile (B = W [d, V] as an MN-major operand); epilogue: E = exp(z - c) in bf16
//                     [rows with a gradient only], per-row partial sums of E, z at the sampled id
//   4. scalar kernel  S, lse = c + log S; ratio, divergence, mask, loss term; row factor g / S; the sampled token's entry
//                     of E becomes E - S (Top-K variants: the K logits per row come from a gather-dot over rows of W^T)
//   5. rescue         rows whose S left the safe range (the sampled token's probability below 2^-60, or non-finite
//                     logits) are packed and go through the two-pass kernels (statistics GEMM with an online maximum,
//                     scalar stage, gradient GEMM writing the finished gradient row into E, row factor 1); normally
//                     there are none and these launches find nothing to do
//   6. dHidden = diag(g / S) (E . W^T)   (A = E, B = W [d,V] K-major), rows scattered back        fp32
//   7. dW = (diag(g / S) hidden)^T . E   (A = scaled packed hidden^T, B = E as MN-major)          fp32
//
// dHidden and dW are d = thousands of columns wide, far more than the 512 accumulator columns of tensor memory, so they
// cannot be accumulated on chip across the vocabulary; the bf16 exponentials E (not the logits) are therefore staged in
// the caller's workspace between steps 3 and 6/7.
#include <mutex>

#include "dppo_common.cuh"
#include "dppo_gemm.cuh"

namespace dppo {

namespace {

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(ptr);
  });
  return fn;
}

// Tensor map of a row-major bf16 matrix [rows, cols] (cols contiguous, leading dimension ld elements) with boxes of
// 64 columns x box_rows rows and the 128-byte swizzle the MMA descriptors expect.  Out-of-range elements read as 0.
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  EncodeFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};       // 64 bf16 = 128 bytes = the swizzle span
  cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of the fp32 output C [rows, cols] (leading dimension ld elements) for the store epilogue: boxes of 32
// columns (128 bytes, the swizzle span) x 32 rows.
bool make_map_c(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld) {
  EncodeFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
  cuuint32_t box[2] = {32u, 32u};
  cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kMaxStreamKSms = 160;                         // SMs the partial-sum buffer of the workspace is sized for
constexpr size_t kStreamKBytes = (size_t)kMaxStreamKSms * gemm::kMaxSegs * gemm::BM * gemm::BN * sizeof(float);

template <int EPI, bool B_MN, int CG>
cudaError_t launch_gemm_cg(const void* A, int64_t lda, const void* B, int64_t ldb, gemm::Params p, cudaStream_t st) {
  using C = gemm::Cfg<CG>;
  CUtensorMap ma, mb, mc;
  if (!make_map(&ma, A, p.M, p.K, lda, gemm::BM)) return cudaErrorInvalidValue;
  if (!(B_MN ? make_map(&mb, B, p.K, p.N, ldb, gemm::BK) : make_map(&mb, B, p.N, p.K, ldb, C::B_COLS))) return cudaErrorInvalidValue;
  // plain outputs (every row of every tile goes to its own place in C) are stored through shared memory by bulk tensor
  // copies when the layout allows a tensor map (16-byte aligned base and row pitch)
  p.tma_store = 0;
  mc = ma;
  if (EPI == gemm::EPI_STORE_F32 && !p.row_map && !p.c_transposed && !p.m_live && !p.sk_part && p.ldc % 4 == 0 &&
      ((uintptr_t)p.C % 16) == 0 && make_map_c(&mc, p.C, p.M, p.N, p.ldc))
    p.tma_store = 1;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  auto kernel = gemm::gemm_tn_kernel<EPI, B_MN, CG>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int64_t ntiles = (int64_t)((p.M + C::TILE_M - 1) / C::TILE_M) * ((p.N + gemm::BN - 1) / gemm::BN);
  const int slots = sms / CG;                               // CTA groups that can be resident at once
  const int groups = (int)(ntiles < slots ? ntiles : slots);
  // the K split of the last wave needs its partial-sum buffer to hold kMaxSegs tiles per group
  if (EPI != gemm::EPI_STORE_F32 || p.c_transposed || p.accumulate || groups < 2 || groups * CG > kMaxStreamKSms) p.sk_part = nullptr;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(groups * CG));
  cfg.blockDim = dim3(gemm::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (CG > 1) ? 1 : 0;
  e = cudaLaunchKernelEx(&cfg, kernel, ma, mb, mc, p);
  if (e != cudaSuccess || !p.sk_part) return e;
  // the tiles of the partial wave: their partial sums are added up in a fixed order
  gemm::gemm_streamk_fixup_kernel<CG><<<dim3((unsigned)(groups - 1), (unsigned)(C::TILE_M / 32)), 256, 0, st>>>(p, groups);
  return cudaGetLastError();
}

// What every GEMM launch of a call takes from the caller's options.
struct GemmOpts {
  int cta_group;                 // 1: one CTA per 128 x 256 tile (cta_group::1); 2: pairs of CTAs per 256 x 256 tile (cta_group::2)
  unsigned long long wait_ns;
  int inject;
};
GemmOpts gemm_opts(const dppo_opts& o) {
  GemmOpts g;
  g.cta_group = (o.gemm_cta_group == 1) ? 1 : 2;
  g.wait_ns = wait_limit_ns(o.wait_limit_us);
  g.inject = o.test_inject;
  return g;
}

// B_MN = false: B is [N, K] with leading dimension ldb; B_MN = true: B is [K, N] with leading dimension ldb.
template <int EPI, bool B_MN = false>
cudaError_t launch_gemm(const GemmOpts& go, const void* A, int64_t lda, const void* B, int64_t ldb, gemm::Params p, cudaStream_t st) {
  if (p.M <= 0 || p.N <= 0 || p.K <= 0) return cudaSuccess;
  p.wait_ns = go.wait_ns;
  p.inject = go.inject;
  return go.cta_group == 2 ? launch_gemm_cg<EPI, B_MN, 2>(A, lda, B, ldb, p, st)
                           : launch_gemm_cg<EPI, B_MN, 1>(A, lda, B, ldb, p, st);
}

// out[c, r] = scale[r] * in[r, c] for bf16 matrices (scale optional: rows at and beyond *n_live count as scale 0);
// 64 x 64 tiles through shared memory, 16-byte global accesses when the layout allows (leading dimensions multiples of
// 8 elements, 16-byte aligned bases), 2-byte accesses at the edges.
__device__ __forceinline__ unsigned short scale_bf16(unsigned short v, float sc) {
  // a zero factor gives an exact zero, whatever the element is (a dropped row may hold non-finite values)
  return sc == 0.f ? (unsigned short)0 : __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float((uint32_t)v << 16) * sc));
}
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* in, int64_t rows, int64_t cols, int64_t ld_in,
                                                             __nv_bfloat16* out, int64_t ld_out, int vec_ok,
                                                             const float* row_scale, const int32_t* n_live) {
  __shared__ unsigned short tile[64][72];                 // [r][c], row pitch 144 bytes (16-byte aligned rows)
  const int64_t r0 = (int64_t)blockIdx.y * 64, c0 = (int64_t)blockIdx.x * 64;
  const int tid = threadIdx.x;
  const unsigned short* src = reinterpret_cast<const unsigned short*>(in);
  unsigned short* dst = reinterpret_cast<unsigned short*>(out);
  const bool interior = vec_ok && r0 + 64 <= rows && c0 + 64 <= cols;
  const int64_t live = n_live ? (int64_t)*n_live : rows;
  if (interior) {
    // 64 rows x 8 vectors of 8 elements: thread -> (row = tid / 8 + 32 * pass, vector = tid % 8)
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      const int r = (tid >> 3) + 32 * pass, v = tid & 7;
      uint4 x = *reinterpret_cast<const uint4*>(src + (r0 + r) * ld_in + c0 + v * 8);
      if (row_scale) {
        const float sc = (r0 + r < live) ? row_scale[r0 + r] : 0.f;
        uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int k = 0; k < 4; ++k)
          w[k] = (uint32_t)scale_bf16((unsigned short)(w[k] & 0xffffu), sc) | ((uint32_t)scale_bf16((unsigned short)(w[k] >> 16), sc) << 16);
        x = make_uint4(w[0], w[1], w[2], w[3]);
      }
      *reinterpret_cast<uint4*>(&tile[r][v * 8]) = x;
    }
    __syncthreads();
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      const int c = (tid >> 3) + 32 * pass, v = tid & 7;     // output row c, 8 consecutive input rows v*8..v*8+7
      unsigned short e[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) e[k] = tile[v * 8 + k][c];
      uint4 x;
      x.x = e[0] | ((uint32_t)e[1] << 16); x.y = e[2] | ((uint32_t)e[3] << 16);
      x.z = e[4] | ((uint32_t)e[5] << 16); x.w = e[6] | ((uint32_t)e[7] << 16);
      *reinterpret_cast<uint4*>(dst + (c0 + c) * ld_out + r0 + v * 8) = x;
    }
  } else {
    const int tx = tid & 63, ty = tid >> 6;
    for (int i = ty; i < 64; i += 4) {
      const int64_t r = r0 + i, c = c0 + tx;
      unsigned short v = (r < rows && c < cols) ? src[r * ld_in + c] : (unsigned short)0;
      if (row_scale) v = scale_bf16(v, (r < rows && r < live) ? row_scale[r] : 0.f);
      tile[i][tx] = v;
    }
    __syncthreads();
    for (int i = ty; i < 64; i += 4) {
      const int64_t c = c0 + i, r = r0 + tx;
      if (c < cols && r < rows) dst[c * ld_out + r] = tile[tx][i];
    }
  }
}

cudaError_t transpose_bf16(const void* in, int64_t rows, int64_t cols, int64_t ld_in, void* out, int64_t ld_out, cudaStream_t st,
                           const float* row_scale = nullptr, const int32_t* n_live = nullptr) {
  if (rows <= 0 || cols <= 0) return cudaSuccess;
  dim3 grid((unsigned)((cols + 63) / 64), (unsigned)((rows + 63) / 64));
  const int vec_ok = (ld_in % 8 == 0) && (ld_out % 8 == 0) && ((uintptr_t)in % 16 == 0) && ((uintptr_t)out % 16 == 0);
  transpose_bf16_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(in), rows, cols, ld_in,
                                              reinterpret_cast<__nv_bfloat16*>(out), ld_out, vec_ok, row_scale, n_live);
  return cudaGetLastError();
}

// cref2[i] = log2(e) * hidden_c[i, :] . W[:, ids[i]]: the reference exponent of packed row i (the logit of its sampled
// token), one warp per row.  The column of W is strided (one 2-byte element per row of W).  Out-of-range ids give 0.
__global__ void __launch_bounds__(256) fused_ref_logit_kernel(const __nv_bfloat16* hc, const __nv_bfloat16* W, int64_t T, int64_t d,
                                                              int64_t V, const int32_t* ids, const int32_t* n_rows, float* cref2) {
  const int lane = threadIdx.x & 31;
  const int64_t i = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (i >= T) return;
  float acc = 0.f;
  const int id = ids[i];
  if (i < (int64_t)*n_rows && id >= 0 && (int64_t)id < V) {
    const unsigned short* h = reinterpret_cast<const unsigned short*>(hc + i * d);
    const unsigned short* w = reinterpret_cast<const unsigned short*>(W) + id;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    int64_t k = lane;
    for (; k + 96 < d; k += 128) {
      a0 = fmaf(__uint_as_float((uint32_t)h[k] << 16), __uint_as_float((uint32_t)w[k * V] << 16), a0);
      a1 = fmaf(__uint_as_float((uint32_t)h[k + 32] << 16), __uint_as_float((uint32_t)w[(k + 32) * V] << 16), a1);
      a2 = fmaf(__uint_as_float((uint32_t)h[k + 64] << 16), __uint_as_float((uint32_t)w[(k + 64) * V] << 16), a2);
      a3 = fmaf(__uint_as_float((uint32_t)h[k + 96] << 16), __uint_as_float((uint32_t)w[(k + 96) * V] << 16), a3);
    }
    for (; k < d; k += 32) a0 = fmaf(__uint_as_float((uint32_t)h[k] << 16), __uint_as_float((uint32_t)w[k * V] << 16), a0);
    acc = (a0 + a1) + (a2 + a3);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) cref2[i] = isfinite(acc) ? acc * kLog2e : 0.f;
}

// z_topk[t, k] = hidden[t, :] . W^T[ids[t, k], :]: the logits at the rollout policy's top-K ids, one warp per (t, k).
// W^T rows are contiguous, so each dot product reads two 2d-byte rows with 16-byte loads (d is a multiple of 8).
__global__ void __launch_bounds__(256) fused_topk_logits_kernel(const __nv_bfloat16* hidden, const __nv_bfloat16* wt, int64_t T,
                                                                int64_t d, int64_t V, const int32_t* ids, int K, float* z_topk,
                                                                float out_scale) {
  const int lane = threadIdx.x & 31;
  const int64_t w = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (w >= T * K) return;
  const int64_t t = w / K;
  const int id = ids[w];
  float acc = 0.f;
  if (id >= 0 && (int64_t)id < V) {
    const uint4* h = reinterpret_cast<const uint4*>(hidden + t * d);
    const uint4* r = reinterpret_cast<const uint4*>(wt + (int64_t)id * d);
    for (int64_t j = lane; j < d / 8; j += 32) {
      const uint4 x = h[j], y = r[j];
      const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc = fmaf(__uint_as_float(xs[i] << 16), __uint_as_float(ys[i] << 16), acc);
        acc = fmaf(__uint_as_float(xs[i] & 0xffff0000u), __uint_as_float(ys[i] & 0xffff0000u), acc);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  // out-of-range ids give 0 here and raise the status bit in the scalar stage (non-finite sums too, when used as reference)
  if (lane == 0) z_topk[w] = (out_scale == 1.f || isfinite(acc)) ? acc * out_scale : 0.f;
}

// Stable two-class partition of the rows (one block): idx = the rows of class 0 in order, then those of class 1;
// pos[t] = the place of row t in idx, or -1 for dropped rows; n[0] = rows of class 0, n[1] = rows of both classes.
//   flag given:  class 0 = rows with flag[t] != 0, everything else dropped
//   otherwise:   class 0 = valid rows (token_mask byte non-zero, or no mask) with adv[t] != 0, class 1 = the other valid rows;
//                rows whose sampled id lies outside [0, V) are dropped (the scalar stage reports them): they must not get
//                a row of exponentials, which would be taken against reference 0 and could overflow
__global__ void __launch_bounds__(1024) fused_partition_rows_kernel(const uint8_t* mask8, const float* adv, const int32_t* flag,
                                                                    const int32_t* ids, int64_t V,
                                                                    int64_t T, int32_t* idx, int32_t* pos, int32_t* n) {
  __shared__ int warp_tot[2][32];
  __shared__ int total[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t per = (T + 1023) / 1024;
  const int64_t t0 = (int64_t)tid * per < T ? (int64_t)tid * per : T, t1 = (t0 + per < T) ? t0 + per : T;
  auto cls = [&](int64_t t) -> int {
    if (flag) return flag[t] != 0 ? 0 : -1;
    if (mask8 && mask8[t] == 0) return -1;
    if (ids[t] < 0 || (int64_t)ids[t] >= V) return -1;
    return adv[t] != 0.f ? 0 : 1;
  };
  int cnt[2] = {0, 0};
  for (int64_t t = t0; t < t1; ++t) { const int c = cls(t); if (c >= 0) ++cnt[c]; }
  int incl[2] = {cnt[0], cnt[1]};
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v0 = __shfl_up_sync(0xffffffffu, incl[0], o), v1 = __shfl_up_sync(0xffffffffu, incl[1], o);
    if (lane >= o) { incl[0] += v0; incl[1] += v1; }
  }
  if (lane == 31) { warp_tot[0][warp] = incl[0]; warp_tot[1][warp] = incl[1]; }
  __syncthreads();
  if (warp < 2) {
    int v = warp_tot[warp][lane], w = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += u; }
    warp_tot[warp][lane] = w - v;                     // exclusive offset of each warp
    if (lane == 31) total[warp] = w;
  }
  __syncthreads();
  if (tid == 0) { n[0] = total[0]; n[1] = total[0] + total[1]; }
  int at[2] = {warp_tot[0][warp] + incl[0] - cnt[0], total[0] + warp_tot[1][warp] + incl[1] - cnt[1]};
  for (int64_t t = t0; t < t1; ++t) {
    const int c = cls(t);
    if (c >= 0) { idx[at[c]] = (int32_t)t; pos[t] = at[c]; ++at[c]; }
    else pos[t] = -1;
  }
}

// dHidden rows of the tokens without a gradient (not valid, or zero advantage): zeros.  The rows with a gradient are
// written by the dHidden GEMM through its row map.
__global__ void __launch_bounds__(256) fused_zero_rows_kernel(const int32_t* pos, const int32_t* n_grad, float* out, int64_t d) {
  const int64_t t = blockIdx.x;
  const int ps = pos[t];
  if (ps >= 0 && ps < *n_grad) return;
  float4* row = reinterpret_cast<float4*>(out + t * d);
  for (int64_t j = threadIdx.x; j < d / 4; j += blockDim.x) row[j] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Two-pass mode: the rows of E from *n_grad up to the end of that block of 64 rows are read by the dW GEMM's last K block
// (against zeros) and written by nobody else unless they belong to valid rows: zeros.
__global__ void __launch_bounds__(256) fused_zero_e_tail_kernel(__nv_bfloat16* E, int64_t lde, const int32_t* n_grad, int64_t T) {
  const int64_t r = (int64_t)*n_grad + blockIdx.x;
  const int64_t end = ((int64_t)*n_grad + 63) / 64 * 64;
  if (r >= end || r >= T) return;
  uint4* row = reinterpret_cast<uint4*>(E + r * lde);
  for (int64_t j = threadIdx.x; j < lde / 8; j += blockDim.x) row[j] = make_uint4(0, 0, 0, 0);
}

// Row i of the compact copies = row idx[i] of the sources for i < *n; after that zeros (zero_fill) or left alone.
struct GatherArgs {
  const int32_t* idx;
  const int32_t* n;
  int64_t d;
  const __nv_bfloat16* src;      // [T, d]
  __nv_bfloat16* dst;            // [T, d]
  const int32_t* ids_in;
  int32_t* ids_out;
  int zero_fill;
};
__global__ void __launch_bounds__(256) fused_gather_rows_kernel(GatherArgs g) {
  const int64_t i = blockIdx.x;
  const bool live = i < (int64_t)*g.n;
  if (!live && !g.zero_fill) return;
  const int64_t t = live ? g.idx[i] : 0;
  const uint4* src = reinterpret_cast<const uint4*>(g.src + t * g.d);
  uint4* dst = reinterpret_cast<uint4*>(g.dst + i * g.d);
  for (int64_t j = threadIdx.x; j < g.d / 8; j += blockDim.x) dst[j] = live ? src[j] : make_uint4(0, 0, 0, 0);
  if (threadIdx.x == 0) g.ids_out[i] = live ? g.ids_in[t] : 0;
}

// What the single-pass scalar stage adds to RowParams.
struct ExpArgs {
  const float* psum;        // [rows, tiles_n] partial sums of exp(z - c) over the entries other than the sampled token's, packed row order
  int tiles_n;
  const float* z_a;         // [rows] z at the sampled id, packed row order
  const float* cref2;       // [rows] c in log2 units, packed row order
  const int32_t* pos;       // [T] packed row of row t, -1: not valid
  const int32_t* n_grad;    // packed rows below *n_grad have a row in E
  const float* z_topk;      // [T, K] or null
  float* row_factor;        // [rows] g / S, packed row order
  int32_t* rescue;          // [T] 1: the row goes through the two-pass kernels
  __nv_bfloat16* E;
  int64_t lde;
  int force_two_pass;       // every valid row goes through the two-pass kernels (psum, z_a, cref2 are not read)
};

// Sums of exp(z - c) above this, or not finite, or not positive, send a row to the two-pass kernels: E and the row
// factor g / S stay far inside the range of bf16 / fp32 for every row that is handled here.
constexpr double kMaxSafeSum = 1.152921504606846976e18;      // 2^60

// One warp per row: S from the forward GEMM's partial sums, then the same scalar stage as the streaming kernels.
__global__ void __launch_bounds__(256) fused_scalar_exp_kernel(RowParams p, ExpArgs x) {
  const int lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= p.T) return;
  const double scale = p.hdr->scale;
  const int64_t ts = (int64_t)x.pos[t];                 // < 0: token_mask says invalid, or the sampled id is out of range
  bool valid = ts >= 0;
  int flags = 0, resc = 0;
  const int a = p.sampled_ids[t];
  if ((!p.token_mask || p.token_mask[t] != 0) && (a < 0 || (int64_t)a >= p.V)) { valid = false; flags = DPPO_STATUS_BAD_SAMPLED_ID; }
  float D = 0.f, r = 0.f, absdiff = 0.f, factor = 0.f;
  int M = 0;
  double g = 0.0;
  if (valid && x.force_two_pass) {
    resc = 1;
  } else if (valid) {
    double S_o = 0.0;                                   // over the entries other than the sampled token's
    for (int i = lane; i < x.tiles_n; i += 32) S_o += (double)x.psum[ts * x.tiles_n + i];
    S_o = warp_sum(S_o);
    const float za = x.z_a[ts];
    const double S = S_o + exp2((double)za * (double)kLog2e - (double)x.cref2[ts]);
    if (!(S > 0.0) || !(S <= kMaxSafeSum)) {
      resc = 1;                                         // outputs of this row are written by the rescue pass
    } else {
      const double lse = ((double)x.cref2[ts] + log2(S)) / (double)kLog2e;
      const double log_other = (S_o > 0.0) ? ((double)x.cref2[ts] + log2(S_o)) / (double)kLog2e : -INFINITY;
      double pi_a;
      int f2 = 0;
      const float* zk = x.z_topk ? x.z_topk + t * (int64_t)p.K : nullptr;
      auto z_at = [&](int, int k) { return k < 0 ? za : zk[k]; };   // sampled id, or position k of the top-K list
      row_scalars_warp(p, t, a, lse, log_other, scale, z_at, D, M, g, r, absdiff, pi_a, f2);
      if (f2) { flags |= f2; D = 0.f; M = 0; g = 0.0; r = 0.f; absdiff = 0.f; }
      else if (g != 0.0) {
        factor = (float)(g / S);
        // the sampled token's entry: g (pi_a - 1) = (g / S) (E_a - S) = -(g / S) S_o
        if (lane == 0 && ts < (int64_t)*x.n_grad) x.E[ts * x.lde + a] = __float2bfloat16_rn((float)(-S_o));
      }
    }
  }
  if (lane == 0) {
    x.rescue[t] = resc;
    if (ts >= 0) x.row_factor[ts] = factor;
    if (!resc) {
      p.divergence[t] = D;
      p.mask[t] = (uint8_t)M;
      p.row_loss[t] = (float)(-g);
      p.row_r[t] = r;
      p.row_absdiff[t] = absdiff;
    }
    if (flags) atomicOr(p.status, flags);
  }
}

// Rescue pass, one warp per flagged row: merge the statistics GEMM's per-tile (max, sum) partials, run the scalar stage
// and leave the coefficients of the gradient epilogue at the row's place among the rescued rows.
struct RescueArgs {
  const int32_t* rescue;    // [T] rows to process
  const int32_t* pos_r;     // [T] place of row t among the rescued rows
  const int32_t* pos_e;     // [T] packed row of row t in E
  const float2* part;       // [rescued rows, tiles_n]
  int tiles_n;
  const float* z_a;         // [rescued rows]
  const float* z_topk;
  float *c2, *sgn, *fix;    // [rescued rows]
  int32_t* p_row_map;       // [rescued rows] row of E the finished gradient row goes to
  float* row_factor;        // [rows of E]
};
__global__ void __launch_bounds__(256) fused_scalar_rescue_kernel(RowParams p, RescueArgs x) {
  const int lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= p.T || !x.rescue[t]) return;
  const double scale = p.hdr->scale;
  const int64_t ts = x.pos_r[t], te = x.pos_e[t];
  int flags = 0;
  const int a = p.sampled_ids[t];
  float D = 0.f, r = 0.f, absdiff = 0.f;
  int M = 0;
  double g = 0.0;
  RowCoef coef;
  coef.c2 = 0.f; coef.sgn = 0.f; coef.fix = 0.f; coef.zero_row = 1;
  float mm = -INFINITY;
  for (int i = lane; i < x.tiles_n; i += 32) mm = fmaxf(mm, x.part[ts * x.tiles_n + i].x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
  double S = 0.0;
  for (int i = lane; i < x.tiles_n; i += 32) {
    const float2 pr = x.part[ts * x.tiles_n + i];
    if (pr.y > 0.f || pr.y != pr.y) S += (double)pr.y * exp((double)pr.x - (double)mm);
  }
  S = warp_sum(S);                                       // over the entries other than the sampled token's
  const float za = x.z_a[ts];
  double lse, log_other;
  combine_lse((double)mm, S, (double)za, lse, log_other);
  if (!isfinite(lse)) {
    flags |= DPPO_STATUS_NONFINITE_ROW;
  } else {
    double pi_a;
    int f2 = 0;
    const float* zk = x.z_topk ? x.z_topk + t * (int64_t)p.K : nullptr;
    auto z_at = [&](int, int k) { return k < 0 ? za : zk[k]; };
    row_scalars_warp(p, t, a, lse, log_other, scale, z_at, D, M, g, r, absdiff, pi_a, f2);
    if (f2) { flags |= f2; D = 0.f; M = 0; g = 0.0; r = 0.f; absdiff = 0.f; }
    else coef = make_coef(g, lse, pi_a);
  }
  if (lane == 0) {
    p.divergence[t] = D;
    p.mask[t] = (uint8_t)M;
    p.row_loss[t] = (float)(-g);
    p.row_r[t] = r;
    p.row_absdiff[t] = absdiff;
    x.c2[ts] = coef.c2;
    x.sgn[ts] = coef.zero_row ? 0.f : coef.sgn;
    x.fix[ts] = coef.fix;
    // the gradient epilogue writes the finished row over the row's exponentials (zeros if g = 0: whatever overflowed
    // there must not meet a later GEMM, not even multiplied by zero)
    x.p_row_map[ts] = (int32_t)te;
    x.row_factor[te] = coef.zero_row ? 0.f : 1.f;
    if (flags) atomicOr(p.status, flags);
  }
}

constexpr size_t kAlign = 256;
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct FusedLayout {
  size_t wt, ht, hc, hr, E, psum, part, z_a, z_ar, z_topk, cref2, factor, c2, sgn, fix, ids_c, ids_r, idx, pos, idx_r, pos_r,
      rescue, rmap, counts, loss_ws, skpart, total;
  int64_t lde, ldt;
  int tiles_n;
};
FusedLayout fused_layout(int64_t T, int64_t d, int64_t V, int K) {
  FusedLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += round_up(bytes ? bytes : 1, kAlign); return o; };
  L.lde = (V + 7) / 8 * 8;
  L.ldt = (T + 7) / 8 * 8;
  L.tiles_n = (int)((V + gemm::BN - 1) / gemm::BN);
  L.wt = take(K > 0 ? (size_t)V * d * 2 : 0);      // W^T is only needed to gather the top-K logits
  L.ht = take((size_t)d * L.ldt * 2);              // packed hidden rows times their row factor, transposed
  L.hc = take((size_t)T * d * 2);                  // hidden rows packed (rows with a gradient, then the other valid rows)
  L.hr = take((size_t)T * d * 2);                  // hidden rows of the rescue pass
  L.E = take((size_t)T * L.lde * 2);
  L.psum = take((size_t)T * L.tiles_n * sizeof(float));
  L.part = take((size_t)T * L.tiles_n * sizeof(float2));
  L.z_a = take((size_t)T * 4);
  L.z_ar = take((size_t)T * 4);
  L.z_topk = take((size_t)T * (K > 0 ? K : 0) * 4);
  L.cref2 = take((size_t)T * 4);
  L.factor = take((size_t)T * 4);
  L.c2 = take((size_t)T * 4);
  L.sgn = take((size_t)T * 4);
  L.fix = take((size_t)T * 4);
  L.ids_c = take((size_t)T * 4);
  L.ids_r = take((size_t)T * 4);
  L.idx = take((size_t)T * 4);
  L.pos = take((size_t)T * 4);
  L.idx_r = take((size_t)T * 4);
  L.pos_r = take((size_t)T * 4);
  L.rescue = take((size_t)T * 4);
  L.rmap = take((size_t)T * 4);
  L.counts = take(4 * sizeof(int32_t));
  L.loss_ws = take(dppo_workspace_bytes(T, V, K, 0));
  L.skpart = take(kStreamKBytes);                  // partial tiles of the dHidden GEMM (K split of its last wave)
  L.total = off;
  return L;
}


// Everything one call of the fused variant needs, for all of its row blocks.
struct FusedCall {
  const __nv_bfloat16* hidden;
  const __nv_bfloat16* W;
  int64_t T, d, V;
  const int32_t* sampled_ids;
  const float* mu_logp;
  const int32_t* topk_ids;
  const float* topk_p;
  const float* adv;
  const uint8_t* token_mask;
  int variant, K;
  float delta;
  dppo_opts o;
  float* loss;
  float* divergence;
  uint8_t* mask;
  float* dHidden;
  float* dW;
  float* stats;
  int32_t* status;
  char* ws;
  FusedLayout L;              // laid out for the rows of one block
  const __nv_bfloat16* wt;    // rows of W^T (Top-K gather, reference logits), or null
  cudaStream_t st;
};

// Steps 1-7 of the file header for the rows [r0, r0 + Tb) of the call.  The scale s and N_valid come from the prelude
// over all rows of the call (already in the workspace header).  `first` / `last`: position of the block in the call;
// the loss reduction adds the block's rows to the totals of the earlier blocks, and dW is overwritten by the first block
// and added to by the later ones (same stream: a fixed order, the result does not depend on timing).
int fused_rows(const FusedCall& c, int64_t r0, int64_t Tb, bool first, bool last) {
  const FusedLayout& L = c.L;
  const int64_t d = c.d, V = c.V;
  const int K = c.K;
  cudaStream_t st = c.st;
  char* ws = c.ws;
  const bool vd = (c.o.lm_head_layout == DPPO_LM_HEAD_VD);      // W and dW given as [V, d]
  const GemmOpts go = gemm_opts(c.o);
  const int32_t* ids_t = c.sampled_ids + r0;
  const uint8_t* tok = c.token_mask ? c.token_mask + r0 : nullptr;
  const int32_t* tk_ids = c.topk_ids ? c.topk_ids + r0 * K : nullptr;

  RowParams p = {};
  p.T = Tb; p.V = V; p.sampled_ids = ids_t; p.mu_logp = c.mu_logp + r0; p.adv = c.adv + r0; p.token_mask = tok;
  p.variant = c.variant; p.K = K; p.topk_ids = tk_ids; p.topk_p = c.topk_p ? c.topk_p + r0 * K : nullptr;
  p.delta = c.delta; p.loss_scale = c.o.loss_scale; p.is_cap = c.o.is_cap; p.eps_low = c.o.eps_low;
  p.divergence = c.divergence + r0; p.mask = c.mask + r0; p.loss = c.loss; p.stats = c.stats; p.status = c.status;
  char* lws = ws + L.loss_ws;
  const size_t per = round_up((size_t)Tb * sizeof(float), kAlign);
  p.hdr = reinterpret_cast<WsHeader*>(lws);
  p.row_loss = reinterpret_cast<float*>(lws + kAlign);
  p.row_r = reinterpret_cast<float*>(lws + kAlign + per);
  p.row_absdiff = reinterpret_cast<float*>(lws + kAlign + 2 * per);

#define DPPO_TRY(call) do { if ((call) != cudaSuccess) return DPPO_ERR_CUDA; } while (0)
  auto F = [&](size_t off) { return reinterpret_cast<float*>(ws + off); };
  auto I = [&](size_t off) { return reinterpret_cast<int32_t*>(ws + off); };
  const __nv_bfloat16* hid = c.hidden + r0 * d;
  const __nv_bfloat16* Wb = c.W;
  __nv_bfloat16* hc = reinterpret_cast<__nv_bfloat16*>(ws + L.hc);
  __nv_bfloat16* E = reinterpret_cast<__nv_bfloat16*>(ws + L.E);
  int32_t* counts = I(L.counts);
  const int32_t *n_grad = counts, *n_valid = counts + 1, *n_resc = counts + 2;
  const unsigned row_warps = (unsigned)((Tb + 7) / 8);
  const int T = (int)Tb;
  // 1. rows with a gradient to come (valid, advantage not zero) first, then the other valid rows
  fused_partition_rows_kernel<<<1, 1024, 0, st>>>(tok, c.adv + r0, nullptr, ids_t, V, Tb, I(L.idx), I(L.pos), counts);
  DPPO_TRY(cudaGetLastError());
  {
    GatherArgs ga = {};
    ga.idx = I(L.idx); ga.n = n_valid; ga.d = d; ga.src = hid; ga.dst = hc; ga.ids_in = ids_t; ga.ids_out = I(L.ids_c);
    ga.zero_fill = 1;
    fused_gather_rows_kernel<<<(unsigned)Tb, 256, 0, st>>>(ga);
    DPPO_TRY(cudaGetLastError());
  }
  const bool two_pass = c.o.fused_two_pass != 0;
  // 2. reference exponent of every packed row
  if (two_pass) {
    fused_zero_e_tail_kernel<<<64, 256, 0, st>>>(E, L.lde, n_grad, Tb);
  } else if (c.wt)      // W^T is there: contiguous rows instead of strided columns (rows past the valid ones are zero: reference 0)
    fused_topk_logits_kernel<<<row_warps, 256, 0, st>>>(hc, c.wt, Tb, d, V, I(L.ids_c), 1, F(L.cref2), kLog2e);
  else
    fused_ref_logit_kernel<<<row_warps, 256, 0, st>>>(hc, Wb, Tb, d, V, I(L.ids_c), n_valid, F(L.cref2));
  DPPO_TRY(cudaGetLastError());
  // 3. forward GEMM: exponentials, their sums, z at the sampled id
  DPPO_TRY(cudaMemsetAsync(F(L.z_a), 0, (size_t)Tb * 4, st));
  gemm::Params g1 = {};
  g1.M = T; g1.N = (int)V; g1.K = (int)d; g1.psum = F(L.psum); g1.z_a = F(L.z_a); g1.ids = I(L.ids_c); g1.cref2 = F(L.cref2);
  g1.P = E; g1.ldp = L.lde; g1.status = c.status; g1.m_live = n_valid; g1.e_live = n_grad;
  if (two_pass) { /* every row is handled by step 5 */ }
  else if (vd) DPPO_TRY((launch_gemm<gemm::EPI_EXP, false>(go, hc, d, Wb, d, g1, st)));     // B = W [V, d], K-major
  else DPPO_TRY((launch_gemm<gemm::EPI_EXP, true>(go, hc, d, Wb, V, g1, st)));         // B = W [d, V], MN-major
  // 4. per-row scalars
  float* z_topk = nullptr;
  if (K > 0) {      // logits at the rollout policy's top-K ids: T x K dot products against rows of W^T
    z_topk = F(L.z_topk);
    fused_topk_logits_kernel<<<(unsigned)((Tb * K + 7) / 8), 256, 0, st>>>(hid, c.wt, Tb, d, V, tk_ids, K, z_topk, 1.f);
    DPPO_TRY(cudaGetLastError());
  }
  {
    ExpArgs x = {};
    x.psum = F(L.psum); x.tiles_n = L.tiles_n; x.z_a = F(L.z_a); x.cref2 = F(L.cref2); x.pos = I(L.pos); x.n_grad = n_grad;
    x.z_topk = z_topk; x.row_factor = F(L.factor); x.rescue = I(L.rescue); x.E = E; x.lde = L.lde;
    x.force_two_pass = two_pass ? 1 : 0;
    fused_scalar_exp_kernel<<<row_warps, 256, 0, st>>>(p, x);
    DPPO_TRY(cudaGetLastError());
  }
  // 5. rescue pass over the rows flagged by the scalar kernel (normally none: the GEMMs then have no tile to process)
  {
    fused_partition_rows_kernel<<<1, 1024, 0, st>>>(nullptr, nullptr, I(L.rescue), nullptr, V, Tb, I(L.idx_r), I(L.pos_r), counts + 2);
    DPPO_TRY(cudaGetLastError());
    GatherArgs ga = {};
    ga.idx = I(L.idx_r); ga.n = n_resc; ga.d = d; ga.src = hid; ga.dst = reinterpret_cast<__nv_bfloat16*>(ws + L.hr);
    ga.ids_in = ids_t; ga.ids_out = I(L.ids_r); ga.zero_fill = 0;
    fused_gather_rows_kernel<<<(unsigned)Tb, 256, 0, st>>>(ga);
    DPPO_TRY(cudaGetLastError());
    DPPO_TRY(cudaMemsetAsync(F(L.z_ar), 0, (size_t)Tb * 4, st));
    gemm::Params gs = {};
    gs.M = T; gs.N = (int)V; gs.K = (int)d; gs.part = reinterpret_cast<float2*>(ws + L.part); gs.z_a = F(L.z_ar);
    gs.ids = I(L.ids_r); gs.status = c.status; gs.m_live = n_resc; gs.allow_empty = 1;
    if (vd) DPPO_TRY((launch_gemm<gemm::EPI_STATS, false>(go, ws + L.hr, d, Wb, d, gs, st)));
    else DPPO_TRY((launch_gemm<gemm::EPI_STATS, true>(go, ws + L.hr, d, Wb, V, gs, st)));
    RescueArgs x = {};
    x.rescue = I(L.rescue); x.pos_r = I(L.pos_r); x.pos_e = I(L.pos);
    x.part = reinterpret_cast<const float2*>(ws + L.part); x.tiles_n = L.tiles_n; x.z_a = F(L.z_ar); x.z_topk = z_topk;
    x.c2 = F(L.c2); x.sgn = F(L.sgn); x.fix = F(L.fix); x.p_row_map = I(L.rmap); x.row_factor = F(L.factor);
    fused_scalar_rescue_kernel<<<row_warps, 256, 0, st>>>(p, x);
    DPPO_TRY(cudaGetLastError());
    gemm::Params gg = {};
    gg.M = T; gg.N = (int)V; gg.K = (int)d; gg.ids = I(L.ids_r); gg.c2 = F(L.c2); gg.sgn = F(L.sgn); gg.fix = F(L.fix);
    gg.P = E; gg.ldp = L.lde; gg.status = c.status; gg.m_live = n_resc; gg.allow_empty = 1; gg.p_row_map = I(L.rmap);
    if (vd) DPPO_TRY((launch_gemm<gemm::EPI_GRAD, false>(go, ws + L.hr, d, Wb, d, gg, st)));
    else DPPO_TRY((launch_gemm<gemm::EPI_GRAD, true>(go, ws + L.hr, d, Wb, V, gg, st)));
  }
  DPPO_TRY(launch_finalize(p, st, first, last));
  // 6. dHidden[idx[i], :] = factor[i] * (E[i, :] . W[d, V]^T) for the rows with a gradient; the other rows are zero.
  //    Few output tiles, very long K: the tiles that do not fill a whole wave of CTA groups are cut along K into
  //    segments that do, and their partial tiles are added up in a fixed order.
  fused_zero_rows_kernel<<<(unsigned)Tb, 256, 0, st>>>(I(L.pos), n_grad, c.dHidden + r0 * d, d);
  DPPO_TRY(cudaGetLastError());
  gemm::Params g3 = {};
  g3.M = T; g3.N = (int)d; g3.K = (int)V; g3.C = c.dHidden + r0 * d; g3.ldc = d; g3.status = c.status;
  g3.m_live = n_grad; g3.row_map = I(L.idx); g3.row_scale = F(L.factor); g3.sk_part = F(L.skpart);
  g3.n_fastest = 1;      // d / 256 tiles along N: the CTAs of a wave then share each 2 V-byte row block of E instead of re-reading it
  if (vd) DPPO_TRY((launch_gemm<gemm::EPI_STORE_F32, true>(go, E, L.lde, Wb, d, g3, st)));     // B = W as [K = V, N = d], MN-major
  else DPPO_TRY(launch_gemm<gemm::EPI_STORE_F32>(go, E, L.lde, Wb, V, g3, st));                // B = W as [N = d, K = V], K-major
  // 7. dW[d, V] (+)= (factor * packed hidden)^T[d, n_grad] . E[n_grad, V]
  DPPO_TRY(transpose_bf16(hc, Tb, d, d, ws + L.ht, L.ldt, st, F(L.factor), n_grad));
  gemm::Params g4 = {};
  g4.M = (int)d; g4.N = (int)V; g4.K = T; g4.C = c.dW; g4.ldc = V; g4.status = c.status; g4.k_live = n_grad;
  g4.accumulate = first ? 0 : 1;
  if (vd) { g4.c_transposed = 1; g4.ldc = d; }      // the same product, stored as dW[V, d]
  DPPO_TRY((launch_gemm<gemm::EPI_STORE_F32, true>(go, ws + L.ht, L.ldt, E, L.lde, g4, st)));   // B = E [T, V], MN-major
#undef DPPO_TRY
  return DPPO_OK;
}

}  // namespace
}  // namespace dppo

extern "C" {

size_t dppo_fused_workspace_bytes(int64_t T, int64_t d, int64_t V, int K) {
  if (T < 0 || d < 1 || V < 1 || K < 0) return 0;
  return dppo::fused_layout(T, d, V, K).total;
}

static int gemm_bf16_checked(bool b_mn, const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K, float* C,
                             int64_t ldc, int32_t* status, const dppo_opts* opts, void* cuda_stream) {
  if (M < 0 || N < 0 || K < 0) return DPPO_ERR_SHAPE;
  if (M == 0 || N == 0) return DPPO_OK;
  if (!A || !B || !C) return DPPO_ERR_NULL;
  if (lda < K || ldb < (b_mn ? N : K) || ldc < N) return DPPO_ERR_STRIDE;
  if (((uintptr_t)A % 16) || ((uintptr_t)B % 16) || (lda % 8) || (ldb % 8) || ((uintptr_t)C % 4)) return DPPO_ERR_ALIGN;
  dppo_opts o = {};
  if (opts) o = *opts;
  if (o.gemm_cta_group < 0 || o.gemm_cta_group > 2 || o.wait_limit_us < 0) return DPPO_ERR_UNSUPPORTED;
  dppo::gemm::Params p = {};
  p.M = M; p.N = N; p.K = K; p.C = C; p.ldc = ldc; p.status = status;
  const dppo::GemmOpts go = dppo::gemm_opts(o);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const cudaError_t e = b_mn ? dppo::launch_gemm<dppo::gemm::EPI_STORE_F32, true>(go, A, lda, B, ldb, p, st)
                             : dppo::launch_gemm<dppo::gemm::EPI_STORE_F32, false>(go, A, lda, B, ldb, p, st);
  return e == cudaSuccess ? DPPO_OK : DPPO_ERR_CUDA;
}

int dppo_gemm_tn_bf16(const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K, float* C, int64_t ldc,
                      int32_t* status, const dppo_opts* opts, void* cuda_stream) {
  return gemm_bf16_checked(false, A, lda, B, ldb, M, N, K, C, ldc, status, opts, cuda_stream);
}

int dppo_gemm_nn_bf16(const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K, float* C, int64_t ldc,
                      int32_t* status, const dppo_opts* opts, void* cuda_stream) {
  return gemm_bf16_checked(true, A, lda, B, ldb, M, N, K, C, ldc, status, opts, cuda_stream);
}

int dppo_fused_lmhead_fwd_bwd(const void* hidden, const void* W, int64_t T, int64_t d, int64_t V,
                              const int32_t* sampled_ids, const float* mu_logp,
                              const int32_t* mu_topk_ids, const float* mu_topk_p, const float* advantages,
                              const uint8_t* token_mask, int variant, int K, float delta, const dppo_opts* opts,
                              float* loss, float* divergence, uint8_t* mask, float* dHidden, float* dW,
                              float* stats, int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  using namespace dppo;
  dppo_opts o = {};
  if (opts) o = *opts;
  if (T < 0 || d < 1 || V < 1 || T > (int64_t)1 << 30 || V > (int64_t)1 << 30 || d > (int64_t)1 << 30) return DPPO_ERR_SHAPE;
  if (variant < DPPO_BINARY_TV || variant > DPPO_GIVEN_D) return DPPO_ERR_VARIANT;
  const bool topk = (variant == DPPO_TOPK_TV || variant == DPPO_TOPK_KL);
  if (!topk) K = 0;
  if (K < 0 || (int64_t)K > V) return DPPO_ERR_SHAPE;
  if (topk && K > 0 && T > 0 && (!mu_topk_ids || !mu_topk_p)) return DPPO_ERR_TOPK;
  if (!loss || !status || !W || !dW) return DPPO_ERR_NULL;
  if (T > 0 && (!hidden || !sampled_ids || !mu_logp || !advantages || !divergence || !mask || !dHidden)) return DPPO_ERR_NULL;
  if (((uintptr_t)hidden % 16) || ((uintptr_t)W % 16) || (d % 8) || (V % 8)) return DPPO_ERR_ALIGN;
  if (((uintptr_t)dHidden % 16) || ((uintptr_t)dW % 16)) return DPPO_ERR_ALIGN;
  if (o.lm_head_layout != DPPO_LM_HEAD_DV && o.lm_head_layout != DPPO_LM_HEAD_VD) return DPPO_ERR_UNSUPPORTED;
  if (o.gemm_cta_group < 0 || o.gemm_cta_group > 2 || o.wait_limit_us < 0 || o.fused_rows_per_block < 0) return DPPO_ERR_UNSUPPORTED;
  if (o.fused_two_pass != 0 && o.fused_two_pass != 1) return DPPO_ERR_UNSUPPORTED;
  const bool vd = (o.lm_head_layout == DPPO_LM_HEAD_VD);
  // row-block mode: the rows are finished block by block and the workspace is sized for one block
  const int64_t Tb_max = (o.fused_rows_per_block > 0 && (int64_t)o.fused_rows_per_block < T) ? (int64_t)o.fused_rows_per_block : T;
  FusedCall c = {};
  c.L = fused_layout(Tb_max, d, V, K);
  if (!workspace || ((uintptr_t)workspace % kAlign) || workspace_bytes < c.L.total) return DPPO_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* ws = reinterpret_cast<char*>(workspace);
  c.hidden = reinterpret_cast<const __nv_bfloat16*>(hidden); c.W = reinterpret_cast<const __nv_bfloat16*>(W);
  c.T = T; c.d = d; c.V = V; c.sampled_ids = sampled_ids; c.mu_logp = mu_logp; c.topk_ids = mu_topk_ids; c.topk_p = mu_topk_p;
  c.adv = advantages; c.token_mask = token_mask; c.variant = variant; c.K = K; c.delta = delta; c.o = o;
  c.loss = loss; c.divergence = divergence; c.mask = mask; c.dHidden = dHidden; c.dW = dW; c.stats = stats; c.status = status;
  c.ws = ws; c.st = st;

  // N_valid and the scale s over ALL rows of the call
  RowParams p0 = {};
  p0.T = T; p0.token_mask = token_mask; p0.loss_scale = o.loss_scale;
  p0.hdr = reinterpret_cast<WsHeader*>(ws + c.L.loss_ws);
  p0.loss = loss; p0.stats = stats; p0.status = status;
  if (launch_prelude(p0, st) != cudaSuccess) return DPPO_ERR_CUDA;
  // dW is written by a GEMM whose K dimension is T: with no rows it is all zero
  if (T == 0) {
    if (cudaMemsetAsync(dW, 0, (size_t)d * V * sizeof(float), st) != cudaSuccess) return DPPO_ERR_CUDA;
    return launch_finalize(p0, st) == cudaSuccess ? DPPO_OK : DPPO_ERR_CUDA;
  }
  // rows of W^T for the gather dot products: W itself when it is stored [V, d]; otherwise a transposed copy, made once
  // per call, when the Top-K lists need it
  c.wt = vd ? c.W : nullptr;
  if (K > 0 && !vd) {
    if (transpose_bf16(W, d, V, V, ws + c.L.wt, d, st) != cudaSuccess) return DPPO_ERR_CUDA;
    c.wt = reinterpret_cast<const __nv_bfloat16*>(ws + c.L.wt);
  }
  for (int64_t r0 = 0; r0 < T; r0 += Tb_max) {
    const int64_t Tb = (T - r0 < Tb_max) ? (T - r0) : Tb_max;
    const int rc = fused_rows(c, r0, Tb, r0 == 0, r0 + Tb >= T);
    if (rc != DPPO_OK) return rc;
  }
  return DPPO_OK;
}

}  // extern "C"
