// Fused LM-head variant of the DPPO loss: logits = hidden x W are produced tile by tile on the tensor cores and
// consumed in the accumulators' epilogue, so the [T, V] logits never exist in memory.
//
//   1. (token mask given) the valid rows of hidden packed together; (Top-K variants) W^T for the gather
//   2. stats GEMM     z-tile = hidden . W-tile (B = W [d, V] as an MN-major operand); epilogue: per-row (max, sum exp)
//                     of the tile, z at the sampled id
//   3. scalar kernel  merge the tiles' partials -> lse; ratio, divergence, mask, loss term, gradient coefficients
//                     (Top-K variants: the K logits per row come from a small gather-dot kernel over rows of W^T)
//   4. packing        rows with a non-zero gradient, in order, packed together (hidden rows, coefficients) and transposed;
//                     their count stays on the device and bounds the tile loops of the three GEMMs below
//   5. grad GEMM      the same tiles again; epilogue: P = dlogits = g (softmax - onehot) in bf16, [rows, V]
//   6. dHidden = P . W^T   (A = P, B = W [d,V] K-major), rows scattered back        fp32
//   7. dW = hidden^T . P   (A = packed hidden^T, B = P as MN-major)                 fp32
//
// dHidden and dW are d = thousands of columns wide, far more than the 512 accumulator columns of tensor memory, so they
// cannot be accumulated on chip across the vocabulary; the bf16 gradient P (not the logits) is therefore staged in the
// caller's workspace between steps 4 and 5/6.
#include <atomic>
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

// 1: one CTA per tile (cta_group::1); 2: pairs of CTAs per 256 x 256 tile (cta_group::2).  Set by dppo_gemm_cta_group.
std::atomic<int> g_cta_group{2};

template <int EPI, bool B_MN, int CG>
cudaError_t launch_gemm_cg(const void* A, int64_t lda, const void* B, int64_t ldb, gemm::Params p, cudaStream_t st) {
  using C = gemm::Cfg<CG>;
  CUtensorMap ma, mb;
  if (!make_map(&ma, A, p.M, p.K, lda, gemm::BM)) return cudaErrorInvalidValue;
  if (!(B_MN ? make_map(&mb, B, p.K, p.N, ldb, gemm::BK) : make_map(&mb, B, p.N, p.K, ldb, C::B_COLS))) return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  auto kernel = gemm::gemm_tn_kernel<EPI, B_MN, CG>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int64_t ntiles = (int64_t)((p.M + C::TILE_M - 1) / C::TILE_M) * ((p.N + gemm::BN - 1) / gemm::BN);
  p.sms = sms;
  int max_splits = 1;
  if (EPI == gemm::EPI_STORE_F32) max_splits = p.splits > 1 ? p.splits : (p.splits < 0 ? 2 : 1);
  // partial sums are added into zeros; with a row map the rows that no tile row maps to stay zero
  if (EPI == gemm::EPI_STORE_F32 && (max_splits > 1 || p.row_map)) {
    cudaError_t ez = cudaMemset2DAsync(p.C, (size_t)p.ldc * sizeof(float), 0, (size_t)p.N * sizeof(float), (size_t)p.M, st);
    if (ez != cudaSuccess) return ez;
  }
  const int64_t nunits = ntiles * max_splits;
  const int slots = sms / CG;                               // CTA groups that can be resident at once
  const int groups = (int)(nunits < slots ? nunits : slots);
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
  return cudaLaunchKernelEx(&cfg, kernel, ma, mb, p);
}

// B_MN = false: B is [N, K] with leading dimension ldb; B_MN = true: B is [K, N] with leading dimension ldb.
template <int EPI, bool B_MN = false>
cudaError_t launch_gemm(const void* A, int64_t lda, const void* B, int64_t ldb, gemm::Params p, cudaStream_t st) {
  if (p.M <= 0 || p.N <= 0 || p.K <= 0) return cudaSuccess;
  return g_cta_group.load() == 2 ? launch_gemm_cg<EPI, B_MN, 2>(A, lda, B, ldb, p, st)
                                 : launch_gemm_cg<EPI, B_MN, 1>(A, lda, B, ldb, p, st);
}

// out[c, r] = in[r, c] for bf16 matrices; 64 x 64 tiles through shared memory, 16-byte global accesses when the
// layout allows (leading dimensions multiples of 8 elements, 16-byte aligned bases), 2-byte accesses at the edges.
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* in, int64_t rows, int64_t cols, int64_t ld_in,
                                                             __nv_bfloat16* out, int64_t ld_out, int vec_ok) {
  __shared__ unsigned short tile[64][72];                 // [r][c], row pitch 144 bytes (16-byte aligned rows)
  const int64_t r0 = (int64_t)blockIdx.y * 64, c0 = (int64_t)blockIdx.x * 64;
  const int tid = threadIdx.x;
  const unsigned short* src = reinterpret_cast<const unsigned short*>(in);
  unsigned short* dst = reinterpret_cast<unsigned short*>(out);
  const bool interior = vec_ok && r0 + 64 <= rows && c0 + 64 <= cols;
  if (interior) {
    // 64 rows x 8 vectors of 8 elements: thread -> (row = tid / 8 + 32 * pass, vector = tid % 8)
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      const int r = (tid >> 3) + 32 * pass, v = tid & 7;
      const uint4 x = *reinterpret_cast<const uint4*>(src + (r0 + r) * ld_in + c0 + v * 8);
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
      tile[i][tx] = (r < rows && c < cols) ? src[r * ld_in + c] : (unsigned short)0;
    }
    __syncthreads();
    for (int i = ty; i < 64; i += 4) {
      const int64_t c = c0 + i, r = r0 + tx;
      if (c < cols && r < rows) dst[c * ld_out + r] = tile[tx][i];
    }
  }
}

cudaError_t transpose_bf16(const void* in, int64_t rows, int64_t cols, int64_t ld_in, void* out, int64_t ld_out, cudaStream_t st) {
  if (rows <= 0 || cols <= 0) return cudaSuccess;
  dim3 grid((unsigned)((cols + 63) / 64), (unsigned)((rows + 63) / 64));
  const int vec_ok = (ld_in % 8 == 0) && (ld_out % 8 == 0) && ((uintptr_t)in % 16 == 0) && ((uintptr_t)out % 16 == 0);
  transpose_bf16_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(in), rows, cols, ld_in,
                                              reinterpret_cast<__nv_bfloat16*>(out), ld_out, vec_ok);
  return cudaGetLastError();
}

// z_topk[t, k] = hidden[t, :] . W^T[ids[t, k], :]: the logits at the rollout policy's top-K ids, one warp per (t, k).
// W^T rows are contiguous, so each dot product reads two 2d-byte rows with 16-byte loads (d is a multiple of 8).
__global__ void __launch_bounds__(256) fused_topk_logits_kernel(const __nv_bfloat16* hidden, const __nv_bfloat16* wt, int64_t T,
                                                                int64_t d, int64_t V, const int32_t* ids, int K, float* z_topk) {
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
  if (lane == 0) z_topk[w] = acc;       // out-of-range ids give 0 here and raise the status bit in the scalar stage
}

// Stable compaction of the rows to keep (one block): idx[i] = i-th kept row, pos[t] = its place in idx or -1, *n = count.
// A row is kept when its token_mask byte is non-zero (mask8 given) or when its gradient sign is non-zero (sgn given).
__global__ void __launch_bounds__(1024) fused_compact_rows_kernel(const uint8_t* mask8, const float* sgn, int64_t T, int32_t* idx,
                                                                  int32_t* pos, int32_t* n) {
  __shared__ int warp_tot[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t per = (T + 1023) / 1024;
  const int64_t t0 = (int64_t)tid * per, t1 = (t0 + per < T) ? t0 + per : T;
  auto keep = [&](int64_t t) { return mask8 ? (mask8[t] != 0) : (sgn[t] != 0.f); };
  int cnt = 0;
  for (int64_t t = t0; t < t1; ++t) cnt += keep(t) ? 1 : 0;
  int incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int v = warp_tot[lane], w = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += u; }
    warp_tot[lane] = w - v;                     // exclusive offset of each warp
    if (lane == 31) *n = w;
  }
  __syncthreads();
  int at = warp_tot[warp] + incl - cnt;
  for (int64_t t = t0; t < t1; ++t) {
    if (keep(t)) { idx[at] = (int32_t)t; pos[t] = at; ++at; }
    else pos[t] = -1;
  }
}

// Row i of the compact copies = row idx[i] of the sources for i < *n, zeros after that (one block per row).
struct GatherArgs {
  const int32_t* idx;
  const int32_t* n;
  int64_t d;
  const __nv_bfloat16* src;      // [T, d]
  __nv_bfloat16* dst;            // [T, d]
  const int32_t* ids_in;
  int32_t* ids_out;
  const float* f_in[3];          // optional per-row floats (null: skipped)
  float* f_out[3];
};
__global__ void __launch_bounds__(256) fused_gather_rows_kernel(GatherArgs g) {
  const int64_t i = blockIdx.x;
  const bool live = i < (int64_t)*g.n;
  const int64_t t = live ? g.idx[i] : 0;
  const uint4* src = reinterpret_cast<const uint4*>(g.src + t * g.d);
  uint4* dst = reinterpret_cast<uint4*>(g.dst + i * g.d);
  for (int64_t j = threadIdx.x; j < g.d / 8; j += blockDim.x) dst[j] = live ? src[j] : make_uint4(0, 0, 0, 0);
  if (threadIdx.x == 0) {
    g.ids_out[i] = live ? g.ids_in[t] : 0;
#pragma unroll
    for (int k = 0; k < 3; ++k)
      if (g.f_in[k]) g.f_out[k][i] = live ? g.f_in[k][t] : 0.f;
  }
}

// One warp per row: merge the stats GEMM's per-tile partials, then the same scalar stage as the streaming kernels.
// `pos` (optional) maps a row to its row in the statistics (rows compacted by the token mask; -1: not there).
__global__ void __launch_bounds__(256) fused_scalar_kernel(RowParams p, const float2* part, int tiles_n, const float* z_a,
                                                           const int32_t* pos, const float* z_topk, float* c2, float* sgn, float* fix) {
  const int lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= p.T) return;
  const double scale = p.hdr->scale;
  bool valid = p.token_mask ? (p.token_mask[t] != 0) : true;
  int flags = 0;
  const int a = p.sampled_ids[t];
  if (valid && (a < 0 || (int64_t)a >= p.V)) { valid = false; flags = DPPO_STATUS_BAD_SAMPLED_ID; }
  float D = 0.f, r = 0.f, absdiff = 0.f;
  int M = 0;
  double g = 0.0;
  RowCoef coef;
  coef.c2 = 0.f; coef.sgn = 0.f; coef.fix = 0.f; coef.zero_row = 1;
  const int64_t ts = pos ? (int64_t)pos[t] : t;       // row of the statistics
  if (ts < 0) valid = false;
  if (valid) {
    float mm = -INFINITY;
    for (int i = lane; i < tiles_n; i += 32) mm = fmaxf(mm, part[ts * tiles_n + i].x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
    double S = 0.0;
    for (int i = lane; i < tiles_n; i += 32) {
      const float2 pr = part[ts * tiles_n + i];
      if (pr.y > 0.f || pr.y != pr.y) S += (double)pr.y * exp((double)pr.x - (double)mm);
    }
    S = warp_sum(S);
    const double lse = (double)mm + log(S);
    if (!isfinite(lse)) {
      flags |= DPPO_STATUS_NONFINITE_ROW;
    } else {
      double pi_a;
      int f2 = 0;
      const float za = z_a[ts];
      const float* zk = z_topk ? z_topk + t * (int64_t)p.K : nullptr;
      auto z_at = [&](int, int k) { return k < 0 ? za : zk[k]; };   // sampled id, or position k of the top-K list
      row_scalars_warp(p, t, a, lse, scale, z_at, D, M, g, r, absdiff, pi_a, f2);
      if (f2) { flags |= f2; D = 0.f; M = 0; g = 0.0; r = 0.f; absdiff = 0.f; }
      else coef = make_coef(g, lse, pi_a);
    }
  }
  if (lane == 0) {
    p.divergence[t] = D;
    p.mask[t] = (uint8_t)M;
    p.row_loss[t] = (float)(-g);
    p.row_r[t] = r;
    p.row_absdiff[t] = absdiff;
    c2[t] = coef.c2;
    sgn[t] = coef.zero_row ? 0.f : coef.sgn;
    fix[t] = coef.fix;
    if (flags) atomicOr(p.status, flags);
  }
}

constexpr size_t kAlign = 256;
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct FusedLayout {
  size_t wt, ht, hc, P, Pt, part, z_a, z_topk, c2, sgn, fix, c2c, sgnc, fixc, ids_c, idx, pos, nlive, loss_ws, total;
  int64_t ldp, ldt;
  int tiles_n;
};
FusedLayout fused_layout(int64_t T, int64_t d, int64_t V, int K) {
  FusedLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += round_up(bytes ? bytes : 1, kAlign); return o; };
  L.ldp = (V + 7) / 8 * 8;
  L.ldt = (T + 7) / 8 * 8;
  L.tiles_n = (int)((V + gemm::BN - 1) / gemm::BN);
  L.wt = take(K > 0 ? (size_t)V * d * 2 : 0);      // W^T is only needed to gather the top-K logits
  L.ht = take((size_t)d * L.ldt * 2);
  L.hc = take((size_t)T * d * 2);                  // hidden rows compacted (valid rows, then rows with a gradient)
  L.P = take((size_t)T * L.ldp * 2);
  L.Pt = 0;
  L.part = take((size_t)T * L.tiles_n * sizeof(float2));
  L.z_a = take((size_t)T * 4);
  L.z_topk = take((size_t)T * (K > 0 ? K : 0) * 4);
  L.c2 = take((size_t)T * 4);
  L.sgn = take((size_t)T * 4);
  L.fix = take((size_t)T * 4);
  L.c2c = take((size_t)T * 4);                     // the same per-row values in compact row order
  L.sgnc = take((size_t)T * 4);
  L.fixc = take((size_t)T * 4);
  L.ids_c = take((size_t)T * 4);
  L.idx = take((size_t)T * 4);
  L.pos = take((size_t)T * 4);
  L.nlive = take(2 * sizeof(int32_t));
  L.loss_ws = take(dppo_workspace_bytes(T));
  L.total = off;
  return L;
}

}  // namespace
}  // namespace dppo

extern "C" {

size_t dppo_fused_workspace_bytes(int64_t T, int64_t d, int64_t V, int K) {
  if (T < 0 || d < 1 || V < 1 || K < 0) return 0;
  return dppo::fused_layout(T, d, V, K).total;
}

int dppo_gemm_cta_group(int cta_group) {
  const int prev = dppo::g_cta_group.load();
  if (cta_group == 1 || cta_group == 2) dppo::g_cta_group.store(cta_group);
  return prev;
}

int dppo_gemm_tn_bf16(const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K, float* C, int64_t ldc,
                      int32_t* status, void* cuda_stream) {
  if (M < 0 || N < 0 || K < 0) return DPPO_ERR_SHAPE;
  if (M == 0 || N == 0) return DPPO_OK;
  if (!A || !B || !C) return DPPO_ERR_NULL;
  if (lda < K || ldb < K || ldc < N) return DPPO_ERR_STRIDE;
  if (((uintptr_t)A % 16) || ((uintptr_t)B % 16) || (lda % 8) || (ldb % 8) || ((uintptr_t)C % 4)) return DPPO_ERR_ALIGN;
  dppo::gemm::Params p = {};
  p.M = M; p.N = N; p.K = K; p.C = C; p.ldc = ldc; p.status = status;
  return dppo::launch_gemm<dppo::gemm::EPI_STORE_F32>(A, lda, B, ldb, p, reinterpret_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? DPPO_OK : DPPO_ERR_CUDA;
}

int dppo_gemm_nn_bf16(const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K, float* C, int64_t ldc,
                      int32_t* status, void* cuda_stream) {
  if (M < 0 || N < 0 || K < 0) return DPPO_ERR_SHAPE;
  if (M == 0 || N == 0) return DPPO_OK;
  if (!A || !B || !C) return DPPO_ERR_NULL;
  if (lda < K || ldb < N || ldc < N) return DPPO_ERR_STRIDE;
  if (((uintptr_t)A % 16) || ((uintptr_t)B % 16) || (lda % 8) || (ldb % 8) || ((uintptr_t)C % 4)) return DPPO_ERR_ALIGN;
  dppo::gemm::Params p = {};
  p.M = M; p.N = N; p.K = K; p.C = C; p.ldc = ldc; p.status = status;
  return dppo::launch_gemm<dppo::gemm::EPI_STORE_F32, true>(A, lda, B, ldb, p, reinterpret_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? DPPO_OK : DPPO_ERR_CUDA;
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
  if (variant < DPPO_BINARY_TV || variant > DPPO_MINIMAL_MASK) return DPPO_ERR_VARIANT;
  const bool topk = (variant == DPPO_TOPK_TV || variant == DPPO_TOPK_KL);
  if (!topk) K = 0;
  if (K < 0 || (int64_t)K > V) return DPPO_ERR_SHAPE;
  if (topk && K > 0 && T > 0 && (!mu_topk_ids || !mu_topk_p)) return DPPO_ERR_TOPK;
  if (!loss || !status || !W || !dW) return DPPO_ERR_NULL;
  if (T > 0 && (!hidden || !sampled_ids || !mu_logp || !advantages || !divergence || !mask || !dHidden)) return DPPO_ERR_NULL;
  if (((uintptr_t)hidden % 16) || ((uintptr_t)W % 16) || (d % 8) || (V % 8)) return DPPO_ERR_ALIGN;
  if (((uintptr_t)dHidden % 16) || ((uintptr_t)dW % 16)) return DPPO_ERR_ALIGN;
  const FusedLayout L = fused_layout(T, d, V, K);
  if (!workspace || ((uintptr_t)workspace % kAlign) || workspace_bytes < L.total) return DPPO_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* ws = reinterpret_cast<char*>(workspace);

  RowParams p = {};
  p.T = T; p.V = V; p.sampled_ids = sampled_ids; p.mu_logp = mu_logp; p.adv = advantages; p.token_mask = token_mask;
  p.variant = variant; p.K = K; p.topk_ids = mu_topk_ids; p.topk_p = mu_topk_p;
  p.delta = delta; p.loss_scale = o.loss_scale; p.is_cap = o.is_cap; p.eps_low = o.eps_low;
  p.divergence = divergence; p.mask = mask; p.loss = loss; p.stats = stats; p.status = status;
  char* lws = ws + L.loss_ws;
  const size_t per = round_up((size_t)T * sizeof(float), kAlign);
  p.hdr = reinterpret_cast<WsHeader*>(lws);
  p.row_loss = reinterpret_cast<float*>(lws + kAlign);
  p.row_r = reinterpret_cast<float*>(lws + kAlign + per);
  p.row_absdiff = reinterpret_cast<float*>(lws + kAlign + 2 * per);

#define DPPO_TRY(call) do { if ((call) != cudaSuccess) return DPPO_ERR_CUDA; } while (0)
  DPPO_TRY(launch_prelude(p, st));
  // dW is written by a GEMM whose K dimension is T: with no rows it is all zero
  if (T == 0) {
    DPPO_TRY(cudaMemsetAsync(dW, 0, (size_t)d * V * sizeof(float), st));
    DPPO_TRY(launch_finalize(p, st));
    return DPPO_OK;
  }
  float2* part = reinterpret_cast<float2*>(ws + L.part);
  float *z_a = reinterpret_cast<float*>(ws + L.z_a), *c2 = reinterpret_cast<float*>(ws + L.c2);
  float *sgn = reinterpret_cast<float*>(ws + L.sgn), *fix = reinterpret_cast<float*>(ws + L.fix);
  int32_t *idx = reinterpret_cast<int32_t*>(ws + L.idx), *pos = reinterpret_cast<int32_t*>(ws + L.pos);
  int32_t *nlive = reinterpret_cast<int32_t*>(ws + L.nlive), *ids_c = reinterpret_cast<int32_t*>(ws + L.ids_c);
  const __nv_bfloat16* hid = reinterpret_cast<const __nv_bfloat16*>(hidden);
  __nv_bfloat16* hc = reinterpret_cast<__nv_bfloat16*>(ws + L.hc);
  auto gather = [&](const int32_t* n, bool coefs) {
    GatherArgs ga = {};
    ga.idx = idx; ga.n = n; ga.d = d; ga.src = hid; ga.dst = hc; ga.ids_in = sampled_ids; ga.ids_out = ids_c;
    if (coefs) {
      ga.f_in[0] = c2; ga.f_in[1] = sgn; ga.f_in[2] = fix;
      ga.f_out[0] = reinterpret_cast<float*>(ws + L.c2c); ga.f_out[1] = reinterpret_cast<float*>(ws + L.sgnc);
      ga.f_out[2] = reinterpret_cast<float*>(ws + L.fixc);
    }
    fused_gather_rows_kernel<<<(unsigned)T, 256, 0, st>>>(ga);
    return cudaGetLastError();
  };
  // 1. W^T for the Top-K gather; with a token mask, the valid rows of hidden packed together for the statistics
  if (K > 0) DPPO_TRY(transpose_bf16(W, d, V, V, ws + L.wt, d, st));
  const void* a_stats = hidden;
  const int32_t* ids_stats = sampled_ids;
  const int32_t *m_stats = nullptr, *pos_stats = nullptr;
  if (token_mask) {
    fused_compact_rows_kernel<<<1, 1024, 0, st>>>(token_mask, nullptr, T, idx, pos, nlive);
    DPPO_TRY(cudaGetLastError());
    DPPO_TRY(gather(nlive, false));
    a_stats = hc; ids_stats = ids_c; m_stats = nlive; pos_stats = pos;
  }
  // 2. statistics of the logits
  DPPO_TRY(cudaMemsetAsync(z_a, 0, (size_t)T * 4, st));
  gemm::Params g1 = {};
  g1.M = (int)T; g1.N = (int)V; g1.K = (int)d; g1.part = part; g1.z_a = z_a; g1.ids = ids_stats; g1.status = status;
  g1.m_live = m_stats;
  DPPO_TRY((launch_gemm<gemm::EPI_STATS, true>(a_stats, d, W, V, g1, st)));      // B = W [d, V], MN-major
  // 3. per-row scalars, loss
  float* z_topk = nullptr;
  if (K > 0) {      // logits at the rollout policy's top-K ids: T x K dot products against rows of W^T
    z_topk = reinterpret_cast<float*>(ws + L.z_topk);
    fused_topk_logits_kernel<<<(unsigned)((T * K + 7) / 8), 256, 0, st>>>(
        hid, reinterpret_cast<const __nv_bfloat16*>(ws + L.wt), T, d, V, mu_topk_ids, K, z_topk);
    DPPO_TRY(cudaGetLastError());
  }
  fused_scalar_kernel<<<(unsigned)((T + 7) / 8), 256, 0, st>>>(p, part, L.tiles_n, z_a, pos_stats, z_topk, c2, sgn, fix);
  DPPO_TRY(cudaGetLastError());
  DPPO_TRY(launch_finalize(p, st));
  // 4. rows whose gradient is zero (invalid, blocked by the mask, zero advantage) drop out of the backward: the rows
  //    that remain are packed together, so the three GEMMs below run over *n_act rows instead of T
  int32_t* n_act = nlive + 1;
  fused_compact_rows_kernel<<<1, 1024, 0, st>>>(nullptr, sgn, T, idx, pos, n_act);
  DPPO_TRY(cudaGetLastError());
  DPPO_TRY(gather(n_act, true));
  DPPO_TRY(transpose_bf16(hc, T, d, d, ws + L.ht, L.ldt, st));
  // 5. gradient with respect to the logits of the packed rows, bf16, [T, ldp] (zero rows from *n_act to the tile's end)
  gemm::Params g2 = {};
  g2.M = (int)T; g2.N = (int)V; g2.K = (int)d; g2.ids = ids_c; g2.c2 = reinterpret_cast<float*>(ws + L.c2c);
  g2.sgn = reinterpret_cast<float*>(ws + L.sgnc); g2.fix = reinterpret_cast<float*>(ws + L.fixc);
  g2.P = reinterpret_cast<__nv_bfloat16*>(ws + L.P); g2.ldp = L.ldp; g2.status = status; g2.m_live = n_act;
  DPPO_TRY((launch_gemm<gemm::EPI_GRAD, true>(hc, d, W, V, g2, st)));
  // 6. dHidden[idx[i], :] = P[i, :] . W[d, V]^T; the other rows stay zero.  Few output tiles, very long K: K is cut in
  //    two when that fills the waves better (two partial sums added into zeros, in either order the same result).
  gemm::Params g3 = {};
  g3.M = (int)T; g3.N = (int)d; g3.K = (int)V; g3.C = dHidden; g3.ldc = d; g3.status = status;
  g3.m_live = n_act; g3.row_map = idx; g3.splits = -1;
  DPPO_TRY(launch_gemm<gemm::EPI_STORE_F32>(ws + L.P, L.ldp, W, V, g3, st));
  // 7. dW[d, V] = packed hidden^T[d, n_act] . P[n_act, V]
  gemm::Params g4 = {};
  g4.M = (int)d; g4.N = (int)V; g4.K = (int)T; g4.C = dW; g4.ldc = V; g4.status = status; g4.k_live = n_act;
  DPPO_TRY((launch_gemm<gemm::EPI_STORE_F32, true>(ws + L.ht, L.ldt, ws + L.P, L.ldp, g4, st)));   // B = P [T, V], MN-major
#undef DPPO_TRY
  return DPPO_OK;
}

}  // extern "C"
