// Exact full-vocabulary divergence between the rollout policy and the trainer policy, streamed from their two logits
// tensors without materialising a probability tensor: per row TV = 1/2 sum |mu - pi|, KL(mu || pi) and the entropy of pi.
// This is what the Binary / Top-K approximations stand in for (App. B) and what makes the "memory-prohibitive" exact
// quantity available as a monitor.  One CTA walks rows blockIdx.x, +gridDim.x, ...:
//   sweep 1  online sums of both rows: (m, S, A = sum e^(z-m) z) for pi and (m', S', B = sum e^(z'-m') (z' - z)) for mu
//            -> lse, entropy = lse - A/S, KL = B/S' - lse' + lse
//   sweep 2  TV = 1/2 sum |e^(z'-lse') - e^(z-lse)|   (second read of both rows, normally from L2)
// One CTA of 512 threads per SM: the row pairs in flight (148 x 608 KB at V = 151936 bf16) then fit in L2 for the
// second read.  With 16-byte aligned rows the sweeps run on whole 8-element vectors, two vectors of each row in flight
// per thread while a third is computed on, and the per-thread reference of the sums only moves when a vector would
// otherwise grow past 2^24.
#include "dppo_common.cuh"
#include "dppo_pipe.cuh"

namespace dppo {
namespace {

constexpr int kThreads = 512;
constexpr float kRefLimit = 1.6e7f;      // a vector's sum of exp(x - reference) may reach this (about 2^24) before the reference moves

struct ExactParams {
  const void* z; const void* zmu;
  int64_t T, V, ld_z, ld_mu;
  const uint8_t* token_mask;
  float* tv; float* kl; float* entropy;      // tv may be null: no second sweep
  int32_t* status;
  unsigned long long wait_ns;
  int inject;
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
  // N values at once against a reference that moves rarely.  The sums are relative to m, whatever m is: the values are
  // first added against the current m; only if that overflows the margin (a partial sum above 2^kRefBits, infinite or
  // NaN) or m is still -inf are they redone against the vector's own maximum.  Weights of entries with e = 0 must not
  // turn 0 * inf into NaN, so they are clamped to the finite range instead of being tested one by one.
  template <int N>
  __device__ __forceinline__ void addN(const float* x, const float* w) {
    const float c = -m * kLog2e;                        // m = -inf: c = +inf, every e below is inf or NaN -> redone
    float ds = 0.f, da = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float e = ex2_approx(fmaf(x[i], kLog2e, c));
      ds += e;
      da = fmaf(e, fminf(fmaxf(w[i], -3.0e38f), 3.0e38f), da);
    }
    if (ds <= kRefLimit) { s += ds; a += da; return; }  // the common case; false for inf and NaN
    float vm = x[0];
#pragma unroll
    for (int i = 1; i < N; ++i) asm("max.NaN.f32 %0, %0, %1;" : "+f"(vm) : "f"(x[i]));
    if (!(vm <= m)) {                                   // a larger maximum, the first finite vector, or NaN
      const float f = ex2_approx((m - vm) * kLog2e);    // m = -inf gives 0
      s *= f; a *= f; m = vm;
    }
    if (m != -INFINITY) {
      const float c2 = -m * kLog2e;
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const float e = ex2_approx(fmaf(x[i], kLog2e, c2));
        s += e;
        a = fmaf(e, (e > 0.f) ? w[i] : 0.f, a);
      }
    }
  }
  __device__ __forceinline__ void add8(const float* x, const float* w) { addN<8>(x, w); }
  // The same on pairs (two fp32 lanes per instruction for the multiply-adds).
  template <int N>
  __device__ __forceinline__ void addN2(const float2* x, const float2* w) {
    const float c = -m * kLog2e;                        // m = -inf: c = +inf, every e below is inf or NaN -> redone
    const float2 l2 = make_float2(kLog2e, kLog2e), c2 = make_float2(c, c);
    float2 ds = make_float2(0.f, 0.f), da = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      const float2 arg = __ffma2_rn(x[i], l2, c2);
      const float2 e = make_float2(ex2_approx(arg.x), ex2_approx(arg.y));
      ds = __fadd2_rn(ds, e);
      da = __ffma2_rn(e, w[i], da);
    }
    const float dsum = ds.x + ds.y, dasum = da.x + da.y;
    // the common case; false for inf and NaN in either sum (an entry far above the reference, or a weight that is not
    // finite: -inf logits give 0 * inf), which the slow path below sorts out entry by entry
    if (dsum <= kRefLimit && fabsf(dasum) <= 3.0e38f) { s += dsum; a += dasum; return; }
    float xs[N], ws[N];
#pragma unroll
    for (int i = 0; i < N / 2; ++i) { xs[2 * i] = x[i].x; xs[2 * i + 1] = x[i].y; ws[2 * i] = w[i].x; ws[2 * i + 1] = w[i].y; }
    float vm = xs[0];
#pragma unroll
    for (int i = 1; i < N; ++i) asm("max.NaN.f32 %0, %0, %1;" : "+f"(vm) : "f"(xs[i]));
    if (!(vm <= m)) {
      const float f = ex2_approx((m - vm) * kLog2e);
      s *= f; a *= f; m = vm;
    }
    if (m == -INFINITY) return;                        // nothing but -inf so far
    const float c3 = -m * kLog2e;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float e = ex2_approx(fmaf(xs[i], kLog2e, c3));
      s += e;
      a = fmaf(e, (e > 0.f) ? ws[i] : 0.f, a);      // e = 0 (a -inf logit) contributes nothing, whatever its weight
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

// The weights z' - z are clamped to +-3e38 inside the sums (see addN), so a rollout probability that meets a trainer
// probability of zero shows up as an astronomically large sum, not as inf: report it as the +inf it stands for.
__device__ __forceinline__ float kl_out(double kl) { return kl > 1e30 ? INFINITY : (float)kl; }

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

// Whole 8-element vectors of an aligned row: raw 16-byte loads first (several in flight), unpacked when used.
template <typename InT> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  uint4 v;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = *reinterpret_cast<const uint4*>(p); }
  __device__ __forceinline__ void unpack(float* o) const {
    o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
    o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
    o[4] = __uint_as_float(v.z << 16); o[5] = __uint_as_float(v.z & 0xffff0000u);
    o[6] = __uint_as_float(v.w << 16); o[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};
template <> struct Raw8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = *reinterpret_cast<const float4*>(p);
    b = *reinterpret_cast<const float4*>(p + 4);
  }
  __device__ __forceinline__ void unpack(float* o) const {
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
  }
};

// Walks the whole 8-element vectors j = tid*8, +kStep, ... of an aligned row pair and hands them to f8(a[8], b[8]) as
// floats; two vector pairs are kept in flight: a buffer is unpacked, refilled with the pair two steps ahead, and only
// then computed on, so that the loads overlap the arithmetic.  Returns the first j that was not processed.
template <typename InT, typename F8>
__device__ __forceinline__ int64_t sweep_vectors(const InT* z, const InT* zm, int64_t V, int64_t j, int64_t step, F8&& f8) {
  Raw8<InT> a0, b0, a1, b1;
  if (j + 8 <= V) { a0.load(z + j); b0.load(zm + j); }
  if (j + step + 8 <= V) { a1.load(z + j + step); b1.load(zm + j + step); }
  for (;;) {
    float a[8], b[8];
    if (j + 8 > V) break;
    a0.unpack(a); b0.unpack(b);
    if (j + 2 * step + 8 <= V) { a0.load(z + j + 2 * step); b0.load(zm + j + 2 * step); }
    f8(a, b);
    j += step;
    if (j + 8 > V) break;
    a1.unpack(a); b1.unpack(b);
    if (j + 2 * step + 8 <= V) { a1.load(z + j + 2 * step); b1.load(zm + j + 2 * step); }
    f8(a, b);
    j += step;
  }
  return j;
}

template <typename InT>
__global__ void __launch_bounds__(kThreads, 1) dppo_exact_kernel(ExactParams p, int vec_ok) {
  __shared__ Acc3 s_pi[kThreads / 32], s_mu[kThreads / 32];
  __shared__ double s_tv[kThreads / 32];
  __shared__ float s_lse[2];
  __shared__ int s_bad;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const InT* Z = reinterpret_cast<const InT*>(p.z);
  const InT* ZM = reinterpret_cast<const InT*>(p.zmu);
  for (int64_t t = blockIdx.x; t < p.T; t += gridDim.x) {
    if (p.token_mask && p.token_mask[t] == 0) {
      if (tid == 0) { if (p.tv) p.tv[t] = 0.f; p.kl[t] = 0.f; p.entropy[t] = 0.f; }
      continue;
    }
    const InT* z = Z + t * p.ld_z;
    const InT* zm = ZM + t * p.ld_mu;
    // ---- sweep 1
    Acc3 api{-INFINITY, 0.f, 0.f}, amu{-INFINITY, 0.f, 0.f};
    constexpr int64_t kStep = (int64_t)kThreads * 8;
    int64_t j = (int64_t)tid * 8;
    if (vec_ok)
      j = sweep_vectors<InT>(z, zm, p.V, j, kStep, [&](float* a, const float* b) {
        api.add8(a, a);
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = b[i] - a[i];
        amu.add8(b, a);
      });
    for (; j < p.V; j += kStep) {
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
    if (warp == 0) {
      // the warps' partials, one per lane, merged by the same fp32 rule as inside a warp; the last step in double
      constexpr int kWarps = kThreads / 32;
      static_assert(kWarps <= 32, "one lane per warp");
      Acc3 xp{-INFINITY, 0.f, 0.f}, xq{-INFINITY, 0.f, 0.f};
      if (lane < kWarps) { xp = s_pi[lane]; xq = s_mu[lane]; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        Acc3 x{__shfl_xor_sync(0xffffffffu, xp.m, o), __shfl_xor_sync(0xffffffffu, xp.s, o), __shfl_xor_sync(0xffffffffu, xp.a, o)};
        Acc3 y{__shfl_xor_sync(0xffffffffu, xq.m, o), __shfl_xor_sync(0xffffffffu, xq.s, o), __shfl_xor_sync(0xffffffffu, xq.a, o)};
        xp.merge(x);
        xq.merge(y);
      }
      if (lane == 0) {
        const double Sp = xp.s, Ap = xp.a, Sq = xq.s, Bq = xq.a;
        const double lse_p = (double)xp.m + log(Sp), lse_q = (double)xq.m + log(Sq);
        const bool ok = isfinite(lse_p) && isfinite(lse_q);
        s_bad = ok ? 0 : 1;
        s_lse[0] = (float)lse_p;
        s_lse[1] = (float)lse_q;
        if (ok) {
          p.entropy[t] = (float)(lse_p - Ap / Sp);
          p.kl[t] = kl_out(Bq / Sq - lse_q + lse_p);
        } else {
          p.entropy[t] = 0.f; p.kl[t] = 0.f;
          if (p.tv) p.tv[t] = 0.f;
          atomicOr(p.status, DPPO_STATUS_NONFINITE_ROW);
        }
      }
    }
    __syncthreads();
    if (s_bad || !p.tv) { __syncthreads(); continue; }
    // ---- sweep 2: total variation with both normalisers known
    const float cp = -s_lse[0] * kLog2e, cq = -s_lse[1] * kLog2e;
    float acc = 0.f;
    j = (int64_t)tid * 8;
    if (vec_ok)
      j = sweep_vectors<InT>(z, zm, p.V, j, kStep, [&](const float* a, const float* b) {
        float part = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) part += fabsf(ex2_approx(fmaf(b[i], kLog2e, cq)) - ex2_approx(fmaf(a[i], kLog2e, cp)));
        acc += part;
      });
    for (; j < p.V; j += kStep) {
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

// ---- 16-byte aligned rows: the same two sweeps fed through a shared-memory ring ------------------------------------
// One producer lane streams the chunks of the row pair (16 KB of each tensor per slot) with bulk asynchronous copies,
// first for sweep 1 (from HBM, kept in L2), then again for sweep 2 (normally from L2), and simply runs ahead as far as
// the ring allows: the consumer warps never wait on global memory, and the copies for sweep 2 are already in flight
// while the row's normalisers are being reduced.  Consumers synchronise among themselves through mbarriers only, so
// every wait in the kernel is bounded (about 2 s; then DPPO_STATUS_WAIT_LIMIT is raised and the CTA leaves).
constexpr int kXChunk = 16384;                       // bytes per tensor per slot
constexpr int kXSlots = 6;
constexpr int kXConsumers = 512;
constexpr int kXWarps = kXConsumers / 32;
constexpr int kXThreads = kXConsumers + 64;          // + producer warp + merger warp (one-sweep mode)
constexpr int kXVec = kXChunk / 16 / kXConsumers;    // 16-byte vectors per thread per chunk and tensor
constexpr int kXMiscBytes = 2048;
static_assert(kXVec * kXConsumers * 16 == kXChunk, "chunk geometry");

struct XMisc {
  unsigned long long full[kXSlots], empty[kXSlots];
  unsigned long long red[2];             // all consumer warps have posted their partials (two sweeps: sweep 1 / sweep 2;
                                         // one sweep: partials buffer 0 / 1)
  unsigned long long red_free[2];        // one sweep: the merger warp has read partials buffer 0 / 1
  Acc3 pi[2][kXWarps], mu[2][kXWarps];   // per-warp partials of a row, two rows deep: without a second sweep a warp may post
                                          // the next row's partials while another still reads this row's
  double tv[kXWarps];
  int abort_flag;
};
static_assert(sizeof(XMisc) <= kXMiscBytes, "misc area");

template <typename InT> struct XVecOf;
template <> struct XVecOf<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void unpack(const uint4& v, float* z) {
    z[0] = __uint_as_float(v.x << 16); z[1] = __uint_as_float(v.x & 0xffff0000u);
    z[2] = __uint_as_float(v.y << 16); z[3] = __uint_as_float(v.y & 0xffff0000u);
    z[4] = __uint_as_float(v.z << 16); z[5] = __uint_as_float(v.z & 0xffff0000u);
    z[6] = __uint_as_float(v.w << 16); z[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};
template <> struct XVecOf<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void unpack(const uint4& v, float* z) {
    z[0] = __uint_as_float(v.x); z[1] = __uint_as_float(v.y); z[2] = __uint_as_float(v.z); z[3] = __uint_as_float(v.w);
  }
};

template <int N>
__device__ __forceinline__ void to_pairs(const float* z, float2* z2) {
#pragma unroll
  for (int i = 0; i < N / 2; ++i) z2[i] = make_float2(z[2 * i], z[2 * i + 1]);
}

// ONE: no TV output: one sweep per row pair, rows finished by the merger warp (launched with kXThreads threads);
// otherwise two sweeps and no merger warp (launched with kXThreads - 32 threads).
template <typename InT, bool ONE>
__global__ void __launch_bounds__(kXThreads, 1) dppo_exact_ring_kernel(ExactParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int N = XVecOf<InT>::N;
  XMisc* misc = reinterpret_cast<XMisc*>(smem + (size_t)kXSlots * 2 * kXChunk);
  const uint32_t slots_base = smem_u32(smem);
  const uint32_t full_base = smem_u32(&misc->full[0]), empty_base = smem_u32(&misc->empty[0]), red_base = smem_u32(&misc->red[0]);
  const uint32_t free_base = smem_u32(&misc->red_free[0]);
  const WaitCtl wc{&misc->abort_flag, p.wait_ns};
  constexpr int passes = ONE ? 1 : 2;       // without a TV output the rows are read once
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int i = 0; i < kXSlots; ++i) { mbar_init(full_base + 8u * i, 1); mbar_init(empty_base + 8u * i, kXWarps); }
    mbar_init(red_base, kXWarps);
    mbar_init(red_base + 8u, kXWarps);
    mbar_init(free_base, 1);
    mbar_init(free_base + 8u, 1);
    misc->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  const uint32_t row_bytes = (uint32_t)(p.V * (int64_t)sizeof(InT));     // launcher guarantees < 2^31
  const int C = (int)((row_bytes + kXChunk - 1) / kXChunk);
  const InT* Z = reinterpret_cast<const InT*>(p.z);
  const InT* ZM = reinterpret_cast<const InT*>(p.zmu);

  if (warp == kXWarps) {
    // ------------------------------------------------------------------ producer (one lane)
    // (test injection: the producer issues nothing, so that every consumer wait of the CTA runs out)
    if (lane == 0 && !(p.inject & DPPO_INJECT_NO_COPIES)) {
      uint64_t keep, drop;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(drop));
      uint32_t it = 0;
      bool ok = true;
      for (int64_t t = blockIdx.x; t < p.T && ok; t += gridDim.x) {
        if (p.token_mask && p.token_mask[t] == 0) continue;
        const char* z = reinterpret_cast<const char*>(Z + t * p.ld_z);
        const char* zm = reinterpret_cast<const char*>(ZM + t * p.ld_mu);
        for (int pass = 0; pass < passes && ok; ++pass) {
          const uint64_t policy = (pass + 1 < passes) ? keep : drop;      // kept in L2 only if it is read again
          for (int c = 0; c < C; ++c, ++it) {
            const uint32_t slot = it % kXSlots, use = it / kXSlots;
            if (use > 0 && !mbar_wait(empty_base + 8u * slot, (use - 1u) & 1u, wc)) { ok = false; break; }
            const uint32_t off = (uint32_t)c * kXChunk;
            const uint32_t bytes = (row_bytes - off) < (uint32_t)kXChunk ? (row_bytes - off) : (uint32_t)kXChunk;
            const uint32_t bar = full_base + 8u * slot, dst = slots_base + slot * (2u * kXChunk);
            mbar_arrive_expect_tx(bar, 2u * bytes);
            bulk_load(dst, z + off, bytes, bar, policy);
            bulk_load(dst + kXChunk, zm + off, bytes, bar, policy);
          }
        }
      }
    }
  } else if (warp == kXWarps + 1) {
    // ------------------------------------------------------------------ merger (one-sweep mode): finishes the rows
    // whose partials the consumer warps have posted, so that those never wait for one another
    if (passes == 1) {
      uint32_t nrow = 0;
      for (int64_t t = blockIdx.x; t < p.T; t += gridDim.x) {
        if (p.token_mask && p.token_mask[t] == 0) continue;
        const uint32_t pb = nrow & 1u, use = nrow >> 1;
        if (!mbar_wait_warp(red_base + 8u * pb, use & 1u, wc)) break;
        Acc3 xp{-INFINITY, 0.f, 0.f}, xq{-INFINITY, 0.f, 0.f};
        if (lane < kXWarps) { xp = misc->pi[pb][lane]; xq = misc->mu[pb][lane]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          Acc3 x{__shfl_xor_sync(0xffffffffu, xp.m, o), __shfl_xor_sync(0xffffffffu, xp.s, o), __shfl_xor_sync(0xffffffffu, xp.a, o)};
          Acc3 y{__shfl_xor_sync(0xffffffffu, xq.m, o), __shfl_xor_sync(0xffffffffu, xq.s, o), __shfl_xor_sync(0xffffffffu, xq.a, o)};
          xp.merge(x);
          xq.merge(y);
        }
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(free_base + 8u * pb);               // the partials are in registers: the buffer may be reused
          const double lse_p = (double)xp.m + log((double)xp.s), lse_q = (double)xq.m + log((double)xq.s);
          if (isfinite(lse_p) && isfinite(lse_q)) {
            p.entropy[t] = (float)(lse_p - (double)xp.a / (double)xp.s);
            p.kl[t] = kl_out((double)xq.a / (double)xq.s - lse_q + lse_p);
          } else {
            p.entropy[t] = 0.f; p.kl[t] = 0.f;
            atomicOr(p.status, DPPO_STATUS_NONFINITE_ROW);
          }
        }
        ++nrow;
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    uint32_t it = 0, nrow = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < p.T && ok; t += gridDim.x) {
      if (p.token_mask && p.token_mask[t] == 0) {
        if (tid == 0) { if (p.tv) p.tv[t] = 0.f; p.kl[t] = 0.f; p.entropy[t] = 0.f; }
        continue;
      }
      // ---- sweep 1
      Acc3 api{-INFINITY, 0.f, 0.f}, amu{-INFINITY, 0.f, 0.f};
      for (int c = 0; c < C && ok; ++c, ++it) {
        const uint32_t slot = it % kXSlots, use = it / kXSlots;
        ok = mbar_wait_warp(full_base + 8u * slot, use & 1u, wc);
        if (!ok) break;
        const uint32_t off = (uint32_t)c * kXChunk;
        const uint32_t nvec = ((row_bytes - off) < (uint32_t)kXChunk ? (row_bytes - off) : (uint32_t)kXChunk) / 16u;
        const uint32_t sa = slots_base + slot * (2u * kXChunk), sb = sa + kXChunk;
        uint4 va[kXVec], vb[kXVec];
#pragma unroll
        for (int k = 0; k < kXVec; ++k) {
          const uint32_t v = (uint32_t)k * kXConsumers + (uint32_t)tid;
          if (v < nvec) { va[k] = lds128(sa + v * 16u); vb[k] = lds128(sb + v * 16u); }
        }
#pragma unroll
        for (int k = 0; k < kXVec; ++k) {
          if ((uint32_t)k * kXConsumers + (uint32_t)tid < nvec) {
            float a[N], b[N];
            XVecOf<InT>::unpack(va[k], a);
            XVecOf<InT>::unpack(vb[k], b);
            float2 a2[N / 2], b2[N / 2];
            to_pairs<N>(a, a2);
            to_pairs<N>(b, b2);
            api.addN2<N>(a2, a2);
            const float2 neg1 = make_float2(-1.f, -1.f);
#pragma unroll
            for (int i = 0; i < N / 2; ++i) a2[i] = __ffma2_rn(a2[i], neg1, b2[i]);      // z' - z
            amu.addN2<N>(b2, a2);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_base + 8u * slot);
      }
      if (!ok) break;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        Acc3 x{__shfl_xor_sync(0xffffffffu, api.m, o), __shfl_xor_sync(0xffffffffu, api.s, o), __shfl_xor_sync(0xffffffffu, api.a, o)};
        Acc3 y{__shfl_xor_sync(0xffffffffu, amu.m, o), __shfl_xor_sync(0xffffffffu, amu.s, o), __shfl_xor_sync(0xffffffffu, amu.a, o)};
        api.merge(x);
        amu.merge(y);
      }
      const uint32_t pb = nrow & 1u;
      if (passes == 1) {
        // One sweep: the warp posts its partials and goes on with the next row; the merger warp finishes the row.
        // Buffer pb was last used two rows ago: wait until the merger has read it.
        bool okw = true;
        if (lane == 0) {
          const uint32_t use = nrow >> 1;
          if (use > 0) okw = mbar_wait(free_base + 8u * pb, (use - 1u) & 1u, wc);
          if (okw) { misc->pi[pb][warp] = api; misc->mu[pb][warp] = amu; mbar_arrive(red_base + 8u * pb); }
        }
        ok = __shfl_sync(0xffffffffu, (int)okw, 0) != 0;
        if (!ok) break;
        ++nrow;
        continue;
      }
      if (lane == 0) { misc->pi[pb][warp] = api; misc->mu[pb][warp] = amu; mbar_arrive(red_base); }
      ok = mbar_wait_warp(red_base, nrow & 1u, wc);
      if (!ok) break;
      // every warp merges the warps' partials for itself (the same fp32 rule, the same order: identical results)
      Acc3 xp{-INFINITY, 0.f, 0.f}, xq{-INFINITY, 0.f, 0.f};
      if (lane < kXWarps) { xp = misc->pi[pb][lane]; xq = misc->mu[pb][lane]; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        Acc3 x{__shfl_xor_sync(0xffffffffu, xp.m, o), __shfl_xor_sync(0xffffffffu, xp.s, o), __shfl_xor_sync(0xffffffffu, xp.a, o)};
        Acc3 y{__shfl_xor_sync(0xffffffffu, xq.m, o), __shfl_xor_sync(0xffffffffu, xq.s, o), __shfl_xor_sync(0xffffffffu, xq.a, o)};
        xp.merge(x);
        xq.merge(y);
      }
      const double lse_p = (double)xp.m + log((double)xp.s), lse_q = (double)xq.m + log((double)xq.s);
      const bool finite = isfinite(lse_p) && isfinite(lse_q);
      if (tid == 0) {
        if (finite) {
          p.entropy[t] = (float)(lse_p - (double)xp.a / (double)xp.s);
          p.kl[t] = kl_out((double)xq.a / (double)xq.s - lse_q + lse_p);
        } else {
          p.entropy[t] = 0.f; p.kl[t] = 0.f;
          atomicOr(p.status, DPPO_STATUS_NONFINITE_ROW);
        }
      }
      // ---- sweep 2 (a non-finite row still drains its chunks: the producer does not know)
      const float cp = -(float)lse_p * kLog2e, cq = -(float)lse_q * kLog2e;
      float acc = 0.f;
      for (int c = 0; c < C && ok; ++c, ++it) {
        const uint32_t slot = it % kXSlots, use = it / kXSlots;
        ok = mbar_wait_warp(full_base + 8u * slot, use & 1u, wc);
        if (!ok) break;
        const uint32_t off = (uint32_t)c * kXChunk;
        const uint32_t nvec = ((row_bytes - off) < (uint32_t)kXChunk ? (row_bytes - off) : (uint32_t)kXChunk) / 16u;
        const uint32_t sa = slots_base + slot * (2u * kXChunk), sb = sa + kXChunk;
        if (finite) {
          uint4 va[kXVec], vb[kXVec];
#pragma unroll
          for (int k = 0; k < kXVec; ++k) {
            const uint32_t v = (uint32_t)k * kXConsumers + (uint32_t)tid;
            if (v < nvec) { va[k] = lds128(sa + v * 16u); vb[k] = lds128(sb + v * 16u); }
          }
#pragma unroll
          for (int k = 0; k < kXVec; ++k) {
            if ((uint32_t)k * kXConsumers + (uint32_t)tid < nvec) {
              float a[N], b[N];
              XVecOf<InT>::unpack(va[k], a);
              XVecOf<InT>::unpack(vb[k], b);
              const float2 l2 = make_float2(kLog2e, kLog2e), cp2 = make_float2(cp, cp), cq2 = make_float2(cq, cq);
              const float2 neg1 = make_float2(-1.f, -1.f);
              float part = 0.f;
#pragma unroll
              for (int i = 0; i < N / 2; ++i) {
                const float2 ea = __ffma2_rn(make_float2(a[2 * i], a[2 * i + 1]), l2, cp2);
                const float2 eb = __ffma2_rn(make_float2(b[2 * i], b[2 * i + 1]), l2, cq2);
                const float2 pa = make_float2(ex2_approx(ea.x), ex2_approx(ea.y)), pb = make_float2(ex2_approx(eb.x), ex2_approx(eb.y));
                const float2 d = __ffma2_rn(pa, neg1, pb);
                part += fabsf(d.x) + fabsf(d.y);
              }
              acc += part;
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_base + 8u * slot);
      }
      if (!ok) break;
      const double d = warp_sum((double)acc);
      if (lane == 0) { misc->tv[warp] = d; mbar_arrive(red_base + 8u); }
      ok = mbar_wait_warp(red_base + 8u, nrow & 1u, wc);
      if (!ok) break;
      if (tid == 0) {
        double tot = 0;
        for (int w = 0; w < kXWarps; ++w) tot += misc->tv[w];
        p.tv[t] = finite ? (float)(0.5 * tot) : 0.f;
      }
      ++nrow;
    }
  }
  __syncwarp();
  if (wc.aborted()) {      // every warp stays until copies that may still be in flight have landed
    if (lane == 0) atomicOr(p.status, DPPO_STATUS_WAIT_LIMIT);
    drain_after_abort();
  }
}

}  // namespace
}  // namespace dppo

extern "C" int dppo_exact_divergence(const void* logits, const void* mu_logits, int64_t T, int64_t V,
                                     int64_t logits_row_stride, int64_t mu_row_stride, int dtype,
                                     const uint8_t* token_mask, float* tv, float* kl, float* entropy,
                                     int32_t* status, const dppo_opts* opts, void* cuda_stream) {
  using namespace dppo;
  if (T < 0 || V < 1) return DPPO_ERR_SHAPE;
  if (dtype != DPPO_F32 && dtype != DPPO_BF16) return DPPO_ERR_DTYPE;
  if (!status) return DPPO_ERR_NULL;
  if (T > 0 && (!logits || !mu_logits || !kl || !entropy)) return DPPO_ERR_NULL;
  if (logits_row_stride < V || mu_row_stride < V) return DPPO_ERR_STRIDE;
  const size_t esz = dtype == DPPO_BF16 ? 2 : 4;
  if (((uintptr_t)logits % esz) || ((uintptr_t)mu_logits % esz)) return DPPO_ERR_ALIGN;
  if (T == 0) return DPPO_OK;
  ExactParams p = {logits, mu_logits, T, V, logits_row_stride, mu_row_stride, token_mask, tv, kl, entropy, status,
                   wait_limit_ns(opts ? opts->wait_limit_us : 0), opts ? opts->test_inject : 0};
  const int vec_ok = ((uintptr_t)logits % 16 == 0) && ((uintptr_t)mu_logits % 16 == 0) &&
                     ((logits_row_stride * esz) % 16 == 0) && ((mu_row_stride * esz) % 16 == 0);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t want = (int64_t)sms;                 // one CTA per SM
  const int grid = (int)(T < want ? T : want);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // aligned rows whose byte length is a multiple of 16 go through the shared-memory ring
  if (vec_ok && (V * (int64_t)esz) % 16 == 0 && V * (int64_t)esz < ((int64_t)1 << 31)) {
    const int smem = kXSlots * 2 * kXChunk + kXMiscBytes;
    cudaError_t e = cudaFuncSetAttribute(dppo_exact_ring_kernel<__nv_bfloat16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(dppo_exact_ring_kernel<__nv_bfloat16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(dppo_exact_ring_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(dppo_exact_ring_kernel<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return DPPO_ERR_CUDA;
    const bool one = (tv == nullptr);
    const int threads = one ? kXThreads : kXThreads - 32;
    if (dtype == DPPO_BF16 && one) dppo_exact_ring_kernel<__nv_bfloat16, true><<<grid, threads, smem, st>>>(p);
    else if (dtype == DPPO_BF16) dppo_exact_ring_kernel<__nv_bfloat16, false><<<grid, threads, smem, st>>>(p);
    else if (one) dppo_exact_ring_kernel<float, true><<<grid, threads, smem, st>>>(p);
    else dppo_exact_ring_kernel<float, false><<<grid, threads, smem, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? DPPO_OK : DPPO_ERR_CUDA;
  }
  if (dtype == DPPO_BF16) dppo_exact_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(p, vec_ok);
  else dppo_exact_kernel<float><<<grid, kThreads, 0, st>>>(p, vec_ok);
  return cudaGetLastError() == cudaSuccess ? DPPO_OK : DPPO_ERR_CUDA;
}
