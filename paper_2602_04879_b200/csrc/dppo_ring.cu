// Row kernel for 16-byte aligned layouts: one persistent CTA per SM streams token rows through a
// ring of shared-memory slots filled by bulk asynchronous copies (TMA, cp.async.bulk) that a
// producer warp issues and mbarriers track.
//
// Per row: sweep 1 consumes the chunks as they land (online max / sum of exponentials); the last
// `nslots` chunks of the row stay resident in the ring, so sweep 2 (the gradient) reads them from
// shared memory; only the head of a row that is longer than the ring is fetched a second time
// (it was loaded with an L2 evict-last hint and normally still sits in L2).  A row that fits in
// the ring is read from HBM exactly once.  The gradient goes out with 128-bit streaming stores.
// While sweep 2 frees slots the producer is already loading the next row into them.
#include "dppo_common.cuh"

namespace dppo {

constexpr int kChunkBytes = 8192;
constexpr int kConsumers = 512;                 // 16 warps; one 16-byte vector per thread per chunk
constexpr int kConsumerWarps = kConsumers / 32;
constexpr int kRingThreads = kConsumers + 32;   // + producer warp
constexpr int kMiscBytes = 1024;                // barriers + reduction scratch
constexpr int kMaxSlots = 28;
static_assert(kChunkBytes == kConsumers * 16, "one vector per consumer thread per chunk");

struct RingMisc {
  unsigned long long full[kMaxSlots];
  unsigned long long empty[kMaxSlots];
  float s_m[kConsumerWarps];
  float s_s[kConsumerWarps];
  RowCoef coef;
  int abort_flag;
};
static_assert(sizeof(RingMisc) <= kMiscBytes, "misc area");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: gives up after ~2 s (or when another thread already gave up) and returns false.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = globaltimer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 0xff) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > 2000000000ull) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void stg128_cs(void* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <typename InT> struct Vec;
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void unpack(const uint4& v, float* z) {
    z[0] = __uint_as_float(v.x << 16); z[1] = __uint_as_float(v.x & 0xffff0000u);
    z[2] = __uint_as_float(v.y << 16); z[3] = __uint_as_float(v.y & 0xffff0000u);
    z[4] = __uint_as_float(v.z << 16); z[5] = __uint_as_float(v.z & 0xffff0000u);
    z[6] = __uint_as_float(v.w << 16); z[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};
template <> struct Vec<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void unpack(const uint4& v, float* z) {
    z[0] = __uint_as_float(v.x); z[1] = __uint_as_float(v.y); z[2] = __uint_as_float(v.z); z[3] = __uint_as_float(v.w);
  }
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Writes N gradient values starting at element j0 of an output row.
template <typename OutT, int N> struct Store;
template <> struct Store<__nv_bfloat16, 8> {
  static __device__ __forceinline__ void run(__nv_bfloat16* row, int64_t j0, const float* v) {
    uint4 o;
    o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
    o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
    stg128_cs(row + j0, o);
  }
};
template <> struct Store<float, 8> {
  static __device__ __forceinline__ void run(float* row, int64_t j0, const float* v) {
    uint4 o0 = {__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3])};
    uint4 o1 = {__float_as_uint(v[4]), __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7])};
    stg128_cs(row + j0, o0);
    stg128_cs(row + j0 + 4, o1);
  }
};
template <> struct Store<float, 4> {
  static __device__ __forceinline__ void run(float* row, int64_t j0, const float* v) {
    uint4 o0 = {__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3])};
    stg128_cs(row + j0, o0);
  }
};

struct RingPos {             // position in the endless sequence of slot uses
  int slot;
  uint32_t phase;
  __device__ __forceinline__ void advance(int nslots, int n = 1) {
    slot += n;
    while (slot >= nslots) { slot -= nslots; phase ^= 1u; }
  }
};

template <typename InT, typename OutT>
__global__ void __launch_bounds__(kRingThreads, 1) dppo_row_ring_kernel(RowParams p, int nslots) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int N = Vec<InT>::N;
  RingMisc* misc = reinterpret_cast<RingMisc*>(smem + (size_t)nslots * kChunkBytes);
  const uint32_t slots_base = smem_u32(smem);
  const uint32_t full_base = smem_u32(&misc->full[0]);
  const uint32_t empty_base = smem_u32(&misc->empty[0]);
  volatile int* abort_flag = &misc->abort_flag;
  const int tid = threadIdx.x;

  if (tid == 0) {
    for (int i = 0; i < nslots; ++i) {
      mbar_init(full_base + 8u * i, 1);
      mbar_init(empty_base + 8u * i, kConsumerWarps);
    }
    misc->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const int64_t row_bytes = p.V * (int64_t)sizeof(InT);
  const int C = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);   // chunks per row
  const int L = C > nslots ? C - nslots : 0;                          // head chunks fetched twice
  const char* logits = reinterpret_cast<const char*>(p.logits);

  if (tid >= kConsumers) {
    // ------------------------------------------------------------------ producer (one lane)
    if (tid == kConsumers) {
      uint64_t pol_keep, pol_stream;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
      RingPos pos{0, 0};
      bool first_lap = true;
      bool ok = true;
      for (int64_t t = blockIdx.x; t < p.T && ok; t += gridDim.x) {
        if (p.token_mask && p.token_mask[t] == 0) continue;
        int a = p.sampled_ids[t];
        if (a < 0 || (int64_t)a >= p.V) continue;
        const char* row = logits + t * p.ld_in * (int64_t)sizeof(InT);
        for (int i = 0; i < C + L; ++i) {
          const int c = (i < C) ? i : i - C;
          if (!first_lap) {
            if (!mbar_wait(empty_base + 8u * pos.slot, pos.phase ^ 1u, abort_flag)) { ok = false; break; }
          }
          const int64_t off = (int64_t)c * kChunkBytes;
          const uint32_t bytes = (uint32_t)((row_bytes - off) < kChunkBytes ? (row_bytes - off) : kChunkBytes);
          const uint32_t bar = full_base + 8u * pos.slot;
          mbar_arrive_expect_tx(bar, bytes);
          bulk_load(slots_base + (uint32_t)pos.slot * kChunkBytes, row + off, bytes, bar,
                    (i < L) ? pol_keep : pol_stream);
          pos.slot += 1;
          if (pos.slot == nslots) { pos.slot = 0; pos.phase ^= 1u; first_lap = false; }
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers (16 warps)
  // A wait that runs out sets abort_flag.  From then on every consumer keeps walking the same
  // control flow (so the named barriers still match) but neither waits nor touches memory, and
  // all of them leave together at the end of the row.
  const int lane = tid & 31, warp = tid >> 5;
  const double scale = p.hdr->scale;
  OutT* dlogits = reinterpret_cast<OutT*>(p.dlogits);
  const uint32_t my_off = (uint32_t)tid * 16u;
  RingPos pos{0, 0};
  bool alive = true;

  for (int64_t t = blockIdx.x; t < p.T; t += gridDim.x) {
    OutT* drow = dlogits + t * p.ld_out;
    bool valid = p.token_mask ? (p.token_mask[t] != 0) : true;
    int a = 0, flags = 0;
    if (valid) {
      a = p.sampled_ids[t];
      if (a < 0 || (int64_t)a >= p.V) { valid = false; flags = DPPO_STATUS_BAD_SAMPLED_ID; }
    }
    if (!valid) {
      float zero[N] = {};
      for (int64_t j0 = (int64_t)tid * N; j0 < p.V; j0 += (int64_t)kConsumers * N) Store<OutT, N>::run(drow, j0, zero);
      if (tid == 0) {
        p.divergence[t] = 0.f; p.mask[t] = 0; p.row_loss[t] = 0.f; p.row_r[t] = 0.f; p.row_absdiff[t] = 0.f;
        if (flags) atomicOr(p.status, flags);
      }
      continue;
    }

    // ---- sweep 1: online (max, sum exp) over the chunks as they land
    float m = -INFINITY, s = 0.f;
    RingPos p1 = pos;
    for (int c = 0; c < C; ++c) {
      if (alive && !mbar_wait(full_base + 8u * p1.slot, p1.phase, abort_flag)) alive = false;
      const int64_t boff = (int64_t)c * kChunkBytes + my_off;
      if (alive && boff < row_bytes) {
        uint4 v = lds128(slots_base + (uint32_t)p1.slot * kChunkBytes + my_off);
        float z[N];
        Vec<InT>::unpack(v, z);
        float vm = z[0];
#pragma unroll
        for (int i = 1; i < N; ++i) vm = fmaxf(vm, z[i]);
        if (vm > m) { s *= ex2_approx((m - vm) * kLog2e); m = vm; }
        const float nm = (m == -INFINITY) ? 0.f : -m * kLog2e;
        float e[N];
#pragma unroll
        for (int i = 0; i < N; ++i) e[i] = ex2_approx(fmaf(z[i], kLog2e, nm));
#pragma unroll
        for (int w = 1; w < N; w <<= 1)
#pragma unroll
          for (int i = 0; i + w < N; i += 2 * w) e[i] += e[i + w];
        s += e[0];
      }
      if (c < L) {                       // head of a long row: give the slot back, it is re-fetched for sweep 2
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_base + 8u * p1.slot);
      }
      p1.advance(nslots);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
      merge_ms(m, s, m2, s2);
    }
    if (lane == 0) { misc->s_m[warp] = m; misc->s_s[warp] = s; }
    consumer_bar();
    const bool dead = (*abort_flag != 0);          // same answer on every consumer here

    // ---- scalar stage (warp 0): lse, ratio, divergence, mask, coefficients
    if (warp == 0) {
      RowCoef coef;
      coef.c2 = 0.f; coef.sgn = 0.f; coef.fix = 0.f; coef.zero_row = 1;
      float D = 0.f, r = 0.f, absdiff = 0.f;
      int M = 0;
      double g = 0.0;
      if (!dead) {
        float mm = -INFINITY;
        for (int w = 0; w < kConsumerWarps; ++w) mm = fmaxf(mm, misc->s_m[w]);
        double S = 0.0;
        for (int w = 0; w < kConsumerWarps; ++w) {
          float sw = misc->s_s[w];
          if (sw > 0.f || sw != sw) S += (double)sw * exp((double)misc->s_m[w] - (double)mm);
        }
        const double lse = (double)mm + log(S);
        if (!isfinite(lse)) {
          flags |= DPPO_STATUS_NONFINITE_ROW;
        } else {
          const InT* zrow = reinterpret_cast<const InT*>(p.logits) + t * p.ld_in;
          double pi_a;
          int f2 = 0;
          auto z_at = [&](int id) { return to_f32<InT>(zrow[id]); };
          row_scalars_warp(p, t, a, lse, scale, z_at, D, M, g, r, absdiff, pi_a, f2);
          if (f2) { flags |= f2; D = 0.f; M = 0; g = 0.0; r = 0.f; absdiff = 0.f; }
          else coef = make_coef(g, lse, pi_a);
        }
      }
      if (lane == 0) {
        misc->coef = coef;
        p.divergence[t] = D;
        p.mask[t] = (uint8_t)M;
        p.row_loss[t] = (float)(-g);
        p.row_r[t] = r;
        p.row_absdiff[t] = absdiff;
        if (flags) atomicOr(p.status, flags);
      }
    }
    consumer_bar();
    const RowCoef coef = misc->coef;
    const uint32_t sign_bit = (coef.sgn < 0.f) ? 0x80000000u : 0u;

    // ---- sweep 2: gradient; resident chunks L..C-1 from the ring, then the re-fetched head 0..L-1
    auto grad_chunk = [&](int c, int slot) {
      const int64_t boff = (int64_t)c * kChunkBytes + my_off;
      if (alive && boff < row_bytes) {
        const int64_t j0 = boff / (int64_t)sizeof(InT);
        float v[N];
        if (coef.zero_row) {
#pragma unroll
          for (int k = 0; k < N; ++k) v[k] = 0.f;
        } else {
          uint4 raw = lds128(slots_base + (uint32_t)slot * kChunkBytes + my_off);
          float z[N];
          Vec<InT>::unpack(raw, z);
#pragma unroll
          for (int k = 0; k < N; ++k)
            v[k] = __uint_as_float(__float_as_uint(ex2_approx(fmaf(z[k], kLog2e, coef.c2))) | sign_bit);
          if ((int64_t)a >= j0 && (int64_t)a < j0 + N) {
#pragma unroll
            for (int k = 0; k < N; ++k)
              if (j0 + k == (int64_t)a) v[k] = coef.fix;
          }
        }
        Store<OutT, N>::run(drow, j0, v);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_base + 8u * slot);
    };
    RingPos p2 = pos;
    p2.advance(nslots, L);
    for (int c = L; c < C; ++c) {
      grad_chunk(c, p2.slot);
      p2.advance(nslots);
    }
    for (int c = 0; c < L; ++c) {                  // p1 points at the first re-fetched chunk
      if (alive && !mbar_wait(full_base + 8u * p1.slot, p1.phase, abort_flag)) alive = false;
      grad_chunk(c, p1.slot);
      p1.advance(nslots);
    }
    pos = p1;                                     // = start + C + L
    consumer_bar();                               // scratch (s_m, coef) is reused by the next row
    if (*abort_flag) break;                       // uniform: written before the barrier
  }
  if (*abort_flag) {
    if (tid == 0) atomicOr(p.status, DPPO_STATUS_WAIT_LIMIT);
    // leave time for bulk copies that may still be in flight towards this CTA's shared memory
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 1000000ull) __nanosleep(1000);
  }
}

static int ring_slots(int dev) {
  int max_smem = 0;
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  int n = (max_smem - kMiscBytes) / kChunkBytes;
  return n > kMaxSlots ? kMaxSlots : n;
}

bool ring_layout_ok(const RowParams& p, int in_dtype, int out_dtype) {
  const int64_t in_sz = (in_dtype == DPPO_BF16) ? 2 : 4, out_sz = (out_dtype == DPPO_BF16) ? 2 : 4;
  if (in_dtype == DPPO_F32 && out_dtype != DPPO_F32) return false;
  if ((p.V * in_sz) % 16 != 0) return false;
  if (((uintptr_t)p.logits) % 16 != 0 || (p.ld_in * in_sz) % 16 != 0) return false;
  if (((uintptr_t)p.dlogits) % 16 != 0 || (p.ld_out * out_sz) % 16 != 0) return false;
  return true;
}

template <typename InT, typename OutT>
static cudaError_t launch_ring_t(const RowParams& p, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int nslots = ring_slots(dev);
  if (nslots < 2) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)nslots * kChunkBytes + kMiscBytes;
  cudaError_t e = cudaFuncSetAttribute(dppo_row_ring_kernel<InT, OutT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = (int)(p.T < sms ? p.T : sms);
  dppo_row_ring_kernel<InT, OutT><<<grid, kRingThreads, smem, st>>>(p, nslots);
  return cudaGetLastError();
}

cudaError_t launch_ring(const RowParams& p, int in_dtype, int out_dtype, cudaStream_t st) {
  if (p.T == 0) return cudaSuccess;
  if (in_dtype == DPPO_F32 && out_dtype == DPPO_F32) return launch_ring_t<float, float>(p, st);
  if (in_dtype == DPPO_BF16 && out_dtype == DPPO_BF16) return launch_ring_t<__nv_bfloat16, __nv_bfloat16>(p, st);
  if (in_dtype == DPPO_BF16 && out_dtype == DPPO_F32) return launch_ring_t<__nv_bfloat16, float>(p, st);
  return cudaErrorInvalidValue;
}

}  // namespace dppo
