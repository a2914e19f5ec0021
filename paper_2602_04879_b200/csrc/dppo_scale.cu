// Row kernel with ONE exponential per logit.  The two-sweep kernel (dppo_ring.cu) evaluates exp twice per element: once
// for the row's normaliser, once more for the gradient when the normaliser is known.  At V = 151 936 the special-function
// pipe is then the busiest unit of the SM and the kernel follows the SM clock instead of the memory system.  Here the
// first sweep measures every logit against a reference that is known before the row starts, the logit of the sampled
// token c_t = z_t[a_t], and writes E_j = exp(z_j - c_t) straight into the gradient's own row of dlogits while it sums
// them (S_t = sum_j E_j >= 1); once S_t is known the gradient is just a rescaling of what is already there,
//
//     dlogits_tj = g_t (softmax_j - [j = a_t]) = (g_t / S_t) E_j          (j != a_t),
//
// so the second sweep reads E back (it was written microseconds earlier and still sits in L2; the write-back cache
// sends the row to HBM once, after the second store), multiplies and stores: no exponential, no logits.  HBM traffic
// stays one read of the logits and one write of the gradient.
//
//   producer lane   bulk copies (TMA) of the row's logits into a shared-memory ring, kept at most one row and a few
//                   chunks ahead of the second sweep, so that the rows between the sweeps fit in L2
//   8 sum warps     E_j = 2^(z_j log2e - c_t log2e), fp32 partial sums, E stored in the gradient's dtype
//   scalar warp     hands c_t to the sum warps one row ahead; afterwards S_t, lse = c_t + log S_t, ratio, divergence,
//                   mask, loss term, and the row factor g_t / S_t for the second sweep
//   producer lane 2 bulk copies of E (from dlogits, i.e. from L2) into a second ring, a row at a time once the sum warps
//                   have finished that row (their stores are fenced towards the async proxy before they say so)
//   8 grad warps    second sweep: dlogits = factor * E, the sampled token's entry set to g_t (pi(a_t) - 1)
//
// A row whose S_t leaves (0, 2^60] (the sampled token has a probability below 2^-60, or the row is not finite) falls
// back to the two-sweep arithmetic inside this kernel: the scalar warp recomputes the normaliser with a running maximum
// from the logits, the grad warps evaluate the exponentials from the logits.  Rare by construction (the sampled token
// was drawn from a policy close to this one); slow but exact.
//
// Layouts: 16-byte aligned rows (as the two-sweep kernel's aligned mode), dlogits not overlapping logits.  With a bf16
// gradient E is rounded to bf16 before it is rescaled and rounded again: the result is within one bf16 unit of the
// correctly rounded gradient.  Every wait is bounded (about 2 s, then DPPO_STATUS_WAIT_LIMIT).
#include <atomic>

#include "dppo_common.cuh"
#include "dppo_pipe.cuh"
#include "dppo_rowtools.cuh"

namespace dppo {
namespace {

constexpr int kSChunk = 16384;
constexpr int kSGroup = 256;                               // threads of the sum group and of the grad group
constexpr int kSWarps = kSGroup / 32;
constexpr int kSVec = kSChunk / 16 / kSGroup;              // 16-byte input vectors per thread per chunk
constexpr int kSThreads = 2 * kSGroup + 96;                // + scalar warp + two producer warps
constexpr int kSMisc = 1024;
constexpr int kSMaxSlots = 14;
constexpr double kMaxSafeSum = 1.152921504606846976e18;    // 2^60
static_assert(kSVec * kSGroup * 16 == kSChunk, "chunk geometry");

struct ScaleCoef {
  float f;        // mode 1: dlogits_j = f * E_j
  float fix;      // value at j = a_t
  float c2, sgn;  // mode 2: dlogits_j = sgn * 2^(z_j log2e + c2)
  int mode;       // 0: zero row; 1: rescale E; 2: evaluate from the logits
};

struct ScaleMisc {
  unsigned long long full[kSMaxSlots], empty[kSMaxSlots];
  unsigned long long cref_full[2], cref_empty[2];          // scalar -> sum: reference exponent of a row
  unsigned long long part_full[2], part_empty[2];          // sum -> scalar: partial sums of a row
  unsigned long long coef_full[2], coef_empty[2];          // scalar -> grad: what to do with the row
  float nref[2];                                           // -c_t * log2e
  float part[2][kSWarps];
  ScaleCoef coef[2];
  int abort_flag;
  unsigned int grad_elems;                                 // elements the second sweep has finished (one lane writes it)
};
static_assert(sizeof(ScaleMisc) <= kSMisc, "misc area");

__device__ __forceinline__ uint64_t keep_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void stg128_keep(void* p, uint4 v) {      // stays in L2: read and overwritten within microseconds
  const uint64_t pol = keep_policy();
  asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol) : "memory");
}

// N exponentials (one input vector) stored in the output dtype at element j0 of the row, to be read back by bulk copies.
template <typename OutT, int N> struct KeepE;
template <> struct KeepE<__nv_bfloat16, 8> {
  static __device__ __forceinline__ void run(__nv_bfloat16* row, uint32_t j0, const float* e) {
    stg128_keep(row + j0, make_uint4(pack_bf16x2(e[0], e[1]), pack_bf16x2(e[2], e[3]), pack_bf16x2(e[4], e[5]), pack_bf16x2(e[6], e[7])));
  }
};
template <> struct KeepE<float, 8> {
  static __device__ __forceinline__ void run(float* row, uint32_t j0, const float* e) {
    stg128_keep(row + j0, make_uint4(__float_as_uint(e[0]), __float_as_uint(e[1]), __float_as_uint(e[2]), __float_as_uint(e[3])));
    stg128_keep(row + j0 + 4, make_uint4(__float_as_uint(e[4]), __float_as_uint(e[5]), __float_as_uint(e[6]), __float_as_uint(e[7])));
  }
};
template <> struct KeepE<float, 4> {
  static __device__ __forceinline__ void run(float* row, uint32_t j0, const float* e) {
    stg128_keep(row + j0, make_uint4(__float_as_uint(e[0]), __float_as_uint(e[1]), __float_as_uint(e[2]), __float_as_uint(e[3])));
  }
};

// log-sum-exp of one row by one warp, with a running maximum, straight from global memory (fallback rows only).
template <typename InT>
__device__ __forceinline__ double warp_row_lse(const InT* zrow, int64_t V) {
  constexpr int N = Vec<InT>::N;
  const int lane = threadIdx.x & 31;
  float m = -INFINITY, s = 0.f;
  for (int64_t j = (int64_t)lane * N; j < V; j += 32 * N) {
    float z[N];
    Vec<InT>::unpack(*reinterpret_cast<const uint4*>(zrow + j), z);       // rows are whole 16-byte vectors
    float vm = z[0];
#pragma unroll
    for (int i = 1; i < N; ++i) asm("max.NaN.f32 %0, %0, %1;" : "+f"(vm) : "f"(z[i]));
    if (!(vm <= m)) { s *= ex2_approx((m - vm) * kLog2e); m = vm; }
    if (m != -INFINITY) {
      const float c = -m * kLog2e;
#pragma unroll
      for (int i = 0; i < N; ++i) s += ex2_approx(fmaf(z[i], kLog2e, c));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    if (m != m || m2 != m2) { m = NAN; s = NAN; } else merge_ms(m, s, m2, s2);
  }
  return (double)m + log((double)s);
}

template <typename InT, typename OutT>
__global__ void __launch_bounds__(kSThreads, 1) dppo_row_scale_kernel(RowParams p, int nslots, int sum_slots, int lead_extra) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int N = Vec<InT>::N;
  ScaleMisc* misc = reinterpret_cast<ScaleMisc*>(smem + (size_t)nslots * kSChunk);
  const uint32_t slots_base = smem_u32(smem);
  const uint32_t full_base = smem_u32(&misc->full[0]), empty_base = smem_u32(&misc->empty[0]);
  const uint32_t cref_full = smem_u32(&misc->cref_full[0]), cref_empty = smem_u32(&misc->cref_empty[0]);
  const uint32_t part_full = smem_u32(&misc->part_full[0]), part_empty = smem_u32(&misc->part_empty[0]);
  const uint32_t coef_full = smem_u32(&misc->coef_full[0]), coef_empty = smem_u32(&misc->coef_empty[0]);
  volatile int* abort_flag = &misc->abort_flag;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int i = 0; i < nslots; ++i) { mbar_init(full_base + 8u * i, 1); mbar_init(empty_base + 8u * i, kSWarps); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(cref_full + 8u * i, 1);
      mbar_init(cref_empty + 8u * i, kSWarps);
      mbar_init(part_full + 8u * i, kSWarps);
      mbar_init(part_empty + 8u * i, 1);
      mbar_init(coef_full + 8u * i, 1);
      mbar_init(coef_empty + 8u * i, kSWarps);
    }
    misc->abort_flag = 0;
    misc->grad_elems = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const uint32_t row_bytes = (uint32_t)(p.V * (int64_t)sizeof(InT));     // launcher guarantees < 2^31
  const int C = (int)((row_bytes + kSChunk - 1) / kSChunk);
  constexpr int NO = 16 / (int)sizeof(OutT);                              // elements of E per 16-byte vector
  const uint32_t erow_bytes = (uint32_t)(p.V * (int64_t)sizeof(OutT));    // launcher guarantees < 2^31
  const int CO = (int)((erow_bytes + kSChunk - 1) / kSChunk);             // chunks of a row of E
  // slots [0, ns_sum) feed the sum warps, [ns_sum, nslots) the grad warps (same split as the two-sweep kernel)
  const int ns_sum = (sum_slots >= 2 && sum_slots <= nslots - 2) ? sum_slots : ((2 * nslots + 3) / 7 < 2 ? 2 : (2 * nslots + 3) / 7);
  const int ns_grad = nslots - ns_sum;
  const int64_t t0 = blockIdx.x, G = gridDim.x;
  const InT* logits = reinterpret_cast<const InT*>(p.logits);
  OutT* dlogits = reinterpret_cast<OutT*>(p.dlogits);

  if (warp == 2 * kSWarps + 1) {
    // ------------------------------------------------------------------ producer of the logits (one lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));    // the logits are read once
      // at most one row and a few chunks ahead of the second sweep: the rows in between wait in L2 as E
      const unsigned int lead_chunks = (unsigned int)(C + (lead_extra >= 2 ? lead_extra : 7));
      const unsigned int lead = lead_chunks * (unsigned int)(kSChunk / sizeof(InT));           // in elements
      volatile unsigned int* follow = &misc->grad_elems;
      RingPos pos{0, 0};
      bool first_lap = true, ok = true;
      unsigned int issued = 0;                                                                  // elements
      int meta = load_meta(p, t0);
      for (int64_t t = t0; t < p.T && ok; t += G) {
        const int meta_next = load_meta(p, t + G);
        if (meta >= 0) {
          const char* row = reinterpret_cast<const char*>(logits + t * p.ld_in);
          for (int c = 0; c < C && ok; ++c) {
            if (issued - *follow >= lead) {
              const unsigned long long w0 = globaltimer_ns();
              while (issued - *follow >= lead) {
                if (*abort_flag) { ok = false; break; }
                if (globaltimer_ns() - w0 > 2000000000ull) { *abort_flag = 1; ok = false; break; }
                __nanosleep(64);
              }
              if (!ok) break;
            }
            if (!first_lap && !mbar_wait(empty_base + 8u * pos.slot, pos.phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t off = (uint32_t)c * kSChunk;
            const uint32_t bytes = (row_bytes - off) < (uint32_t)kSChunk ? (row_bytes - off) : (uint32_t)kSChunk;
            issued += bytes / (uint32_t)sizeof(InT);
            const uint32_t bar = full_base + 8u * pos.slot;
            mbar_arrive_expect_tx(bar, bytes);
            bulk_load(slots_base + (uint32_t)pos.slot * kSChunk, row + off, bytes, bar, policy);
            if (++pos.slot == ns_sum) { pos.slot = 0; pos.phase ^= 1u; first_lap = false; }
          }
        }
        meta = meta_next;
      }
    }
  } else if (warp == 2 * kSWarps + 2) {
    // ------------------------------------------------------------------ producer of E (one lane): dlogits -> grad ring
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));    // about to be overwritten
      RingPos pos{0, 0};
      bool first_lap = true, ok = true;
      uint32_t vrow = 0;
      int meta = load_meta(p, t0);
      for (int64_t t = t0; t < p.T && ok; t += G) {
        const int meta_next = load_meta(p, t + G);
        if (meta >= 0) {
          // the row's E is complete when all sum warps have posted their partial sums (the same barrier the scalar warp
          // waits on; this lane cannot fall two rows behind it, see the lead above)
          const uint32_t b = vrow & 1u;
          if (!mbar_wait(part_full + 8u * b, (vrow >> 1) & 1u, abort_flag)) break;
          asm volatile("fence.proxy.async;" ::: "memory");
          const char* row = reinterpret_cast<const char*>(dlogits + t * p.ld_out);
          for (int c = 0; c < CO; ++c) {
            const int slot = ns_sum + pos.slot;
            if (!first_lap && !mbar_wait(empty_base + 8u * slot, pos.phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t off = (uint32_t)c * kSChunk;
            const uint32_t bytes = (erow_bytes - off) < (uint32_t)kSChunk ? (erow_bytes - off) : (uint32_t)kSChunk;
            const uint32_t bar = full_base + 8u * slot;
            mbar_arrive_expect_tx(bar, bytes);
            bulk_load(slots_base + (uint32_t)slot * kSChunk, row + off, bytes, bar, policy);
            if (++pos.slot == ns_grad) { pos.slot = 0; pos.phase ^= 1u; first_lap = false; }
          }
          ++vrow;
        }
        meta = meta_next;
      }
    }
  } else if (warp < kSWarps) {
    // ------------------------------------------------------------------ sum warps: first sweep
    const uint32_t gtid = (uint32_t)tid;
    RingPos pos{0, 0};
    uint32_t vrow = 0;
    int meta = load_meta(p, t0);
    for (int64_t t = t0; t < p.T; t += G) {
      const int meta_next = load_meta(p, t + G);
      if (__shfl_sync(0xffffffffu, *abort_flag, 0)) break;
      if (meta >= 0) {
        const uint32_t b = vrow & 1u;
        const bool have_ref = mbar_wait_warp(cref_full + 8u * b, (vrow >> 1) & 1u, abort_flag);
        const float nm = misc->nref[b];
        __syncwarp();
        if (lane == 0 && have_ref) mbar_arrive(cref_empty + 8u * b);
        OutT* erow = dlogits + t * p.ld_out;
        const float2 l2 = make_float2(kLog2e, kLog2e), nm2 = make_float2(nm, nm);
        float s = 0.f;
        for (int c = 0; c < C; ++c) {
          const bool ok = have_ref && mbar_wait_warp(full_base + 8u * pos.slot, pos.phase, abort_flag);
          const uint32_t cbase = (uint32_t)c * kSChunk;
          const uint32_t sbase = slots_base + (uint32_t)pos.slot * kSChunk;
          if (ok) {
            if (cbase + (uint32_t)kSChunk <= row_bytes) {
              // whole chunk, straight line: loads, kSVec x N independent exponentials, stores
              uint4 v[kSVec];
#pragma unroll
              for (int k = 0; k < kSVec; ++k) v[k] = lds128(sbase + ((uint32_t)k * kSGroup + gtid) * 16u);
              float2 acc = make_float2(0.f, 0.f);
#pragma unroll
              for (int k = 0; k < kSVec; ++k) {
                float z[N], e[N];
                Vec<InT>::unpack(v[k], z);
#pragma unroll
                for (int i = 0; i < N; i += 2) {
                  const float2 arg = __ffma2_rn(make_float2(z[i], z[i + 1]), l2, nm2);
                  e[i] = ex2_approx(arg.x);
                  e[i + 1] = ex2_approx(arg.y);
                  acc = __fadd2_rn(acc, make_float2(e[i], e[i + 1]));
                }
                KeepE<OutT, N>::run(erow, (cbase / (uint32_t)sizeof(InT)) + ((uint32_t)k * kSGroup + gtid) * N, e);
              }
              s += acc.x + acc.y;
            } else {
#pragma unroll 1
              for (int k = 0; k < kSVec; ++k) {
                const uint32_t off = ((uint32_t)k * kSGroup + gtid) * 16u;
                if (cbase + off < row_bytes) {
                  float z[N], e[N];
                  Vec<InT>::unpack(lds128(sbase + off), z);
                  float vs = 0.f;
#pragma unroll
                  for (int i = 0; i < N; ++i) { e[i] = ex2_approx(fmaf(z[i], kLog2e, nm)); vs += e[i]; }
                  s += vs;
                  KeepE<OutT, N>::run(erow, (cbase + off) / (uint32_t)sizeof(InT), e);
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_base + 8u * pos.slot);
          pos.advance(ns_sum);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        asm volatile("fence.proxy.async;" ::: "memory");      // this lane's stores of E, towards the bulk copies that read them
        __syncwarp();                             // every lane's stores of E are ordered before lane 0's arrival below
        if (lane == 0) {
          bool ok = true;
          if (vrow >= 2) ok = mbar_wait(part_empty + 8u * b, ((vrow >> 1) & 1u) ^ 1u, abort_flag);
          if (ok) {
            misc->part[b][warp] = s;
            mbar_arrive(part_full + 8u * b);      // release: the row's stores of E are ordered before it
          }
        }
        ++vrow;
      }
      meta = meta_next;
    }
  } else if (warp < 2 * kSWarps) {
    // ------------------------------------------------------------------ grad warps: second sweep
    const uint32_t gtid = (uint32_t)(tid - kSGroup);
    RingPos pos{0, 0};
    uint32_t vrow = 0;
    unsigned int elems_done = 0;
    int meta = load_meta(p, t0);
    for (int64_t t = t0; t < p.T; t += G) {
      const int meta_next = load_meta(p, t + G);
      if (__shfl_sync(0xffffffffu, *abort_flag, 0)) break;
      OutT* drow = dlogits + t * p.ld_out;
      if (meta < 0) {
        const float zero[NO] = {};
        for (uint32_t j0 = gtid * NO; j0 < (uint32_t)p.V; j0 += kSGroup * NO) Store<OutT, NO>::run(drow, j0, zero);
      } else {
        const uint32_t b = vrow & 1u;
        const bool have = mbar_wait_warp(coef_full + 8u * b, (vrow >> 1) & 1u, abort_flag);
        ScaleCoef coef = misc->coef[b];
        __syncwarp();
        if (lane == 0 && have) mbar_arrive(coef_empty + 8u * b);
        if (!have) coef.mode = 0;
        const uint32_t a = (uint32_t)meta;
        const InT* zrow = logits + t * p.ld_in;
        const uint32_t sign2 = (coef.sgn < 0.f) ? 0x80008000u : 0u;
        for (int c = 0; c < CO; ++c) {
          const int slot = ns_sum + pos.slot;
          const bool ok = mbar_wait_warp(full_base + 8u * slot, pos.phase, abort_flag);
          const uint32_t cbase = (uint32_t)c * kSChunk;
          const uint32_t sbase = slots_base + (uint32_t)slot * kSChunk;
          if (ok) {
            const uint32_t e0 = cbase / (uint32_t)sizeof(OutT);                       // first element of the chunk
            const bool has_a = (a - e0) < (uint32_t)(kSChunk / sizeof(OutT));         // warp-uniform
            if (coef.mode == 1 && cbase + (uint32_t)kSChunk <= erow_bytes && !has_a) {
              // straight-line path: loads, multiplies, stores
              uint4 raw[kSVec];
#pragma unroll
              for (int k = 0; k < kSVec; ++k) raw[k] = lds128(sbase + ((uint32_t)k * kSGroup + gtid) * 16u);
#pragma unroll
              for (int k = 0; k < kSVec; ++k) {
                float v[NO];
                Vec<OutT>::unpack(raw[k], v);
#pragma unroll
                for (int i = 0; i < NO; ++i) v[i] *= coef.f;
                Store<OutT, NO>::run(drow, e0 + ((uint32_t)k * kSGroup + gtid) * NO, v);
              }
            } else {
#pragma unroll 1
              for (int k = 0; k < kSVec; ++k) {
                const uint32_t off = ((uint32_t)k * kSGroup + gtid) * 16u;
                if (cbase + off < erow_bytes) {
                  const uint32_t j0 = (cbase + off) / (uint32_t)sizeof(OutT);
                  float v[NO];
                  uint32_t flip = 0u;
                  if (coef.mode == 1) {
                    Vec<OutT>::unpack(lds128(sbase + off), v);
#pragma unroll
                    for (int i = 0; i < NO; ++i) v[i] *= coef.f;
                  } else if (coef.mode == 2) {                    // fallback row: from the logits, with the exponential
#pragma unroll
                    for (int i = 0; i < NO; ++i) v[i] = ex2_approx(fmaf(to_f32<InT>(zrow[j0 + i]), kLog2e, coef.c2));
                    flip = sign2;
                  } else {
#pragma unroll
                    for (int i = 0; i < NO; ++i) v[i] = 0.f;
                  }
                  if (coef.mode != 0 && a - j0 < (uint32_t)NO) {   // the sampled token's entry is g (pi(a) - 1)
#pragma unroll
                    for (int i = 0; i < NO; ++i)
                      if (j0 + i == a) v[i] = flip ? coef.fix * coef.sgn : coef.fix;      // a flipped store flips it back
                  }
                  Store<OutT, NO>::run(drow, j0, v, flip);
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_base + 8u * slot);
          const uint32_t cb = (erow_bytes - cbase) < (uint32_t)kSChunk ? (erow_bytes - cbase) : (uint32_t)kSChunk;
          elems_done += cb / (uint32_t)sizeof(OutT);
          if (tid == kSGroup) *(volatile unsigned int*)&misc->grad_elems = elems_done;
          pos.advance(ns_grad);
        }
        ++vrow;
      }
      meta = meta_next;
    }
  } else {
    // ------------------------------------------------------------------ scalar warp
    const double scale = p.hdr->scale;
    const bool topk = (p.variant == DPPO_TOPK_TV || p.variant == DPPO_TOPK_KL) && p.K > 0;
    // the reference of a row goes to the sum warps one valid row ahead of the row whose sums are awaited here
    int64_t t_ref = t0;            // next row whose reference has not been posted
    uint32_t v_ref = 0;            // its index among the valid rows
    float za_q[2] = {0.f, 0.f};    // z[a_t] of the two rows in flight
    bool alive = true;
    auto post_next_ref = [&]() {
      while (t_ref < p.T && load_meta(p, t_ref) < 0) t_ref += G;
      if (t_ref >= p.T || !alive) return;
      const int a = p.sampled_ids[t_ref];
      const float z_a = to_f32<InT>(logits[t_ref * p.ld_in + a]);
      const uint32_t b = v_ref & 1u;
      if (lane == 0) {
        bool ok = true;
        if (v_ref >= 2) ok = mbar_wait(cref_empty + 8u * b, ((v_ref >> 1) & 1u) ^ 1u, abort_flag);
        if (ok) {
          misc->nref[b] = -z_a * kLog2e;
          mbar_arrive(cref_full + 8u * b);
        }
      }
      if (b == 0) za_q[0] = z_a; else za_q[1] = z_a;
      ++v_ref;
      t_ref += G;
    };
    post_next_ref();
    uint32_t vrow = 0;
    int meta = load_meta(p, t0);
    for (int64_t t = t0; t < p.T; t += G) {
      const int meta_next = load_meta(p, t + G);
      if (__shfl_sync(0xffffffffu, *abort_flag, 0)) { alive = false; break; }
      int flags = (meta == -2) ? DPPO_STATUS_BAD_SAMPLED_ID : 0;
      float D = 0.f, r = 0.f, absdiff = 0.f;
      int M = 0;
      double g = 0.0;
      if (meta >= 0) {
        const int a = meta;
        const uint32_t b = vrow & 1u;
        const float z_a = (b == 0) ? za_q[0] : za_q[1];
        post_next_ref();                                  // the next valid row may start while this one is finished
        const InT* zrow = logits + t * p.ld_in;
        // Top-K variants: this lane's list entries and their logits, fetched before the wait (see dppo_ring.cu)
        constexpr int kPre = 4;
        float zk_pre[kPre] = {0.f, 0.f, 0.f, 0.f}, pm_pre[kPre] = {0.f, 0.f, 0.f, 0.f};
        int id_pre[kPre] = {-1, -1, -1, -1};
        if (topk) {
          const int32_t* ids = p.topk_ids + t * (int64_t)p.K;
          const float* ps = p.topk_p + t * (int64_t)p.K;
#pragma unroll
          for (int i = 0; i < kPre; ++i) {
            const int k = lane + 32 * i;
            if (k < p.K) { id_pre[i] = ids[k]; pm_pre[i] = ps[k]; }
          }
#pragma unroll
          for (int i = 0; i < kPre; ++i)
            if (id_pre[i] >= 0 && (int64_t)id_pre[i] < p.V) zk_pre[i] = to_f32<InT>(zrow[id_pre[i]]);
        }
        const bool have = mbar_wait_warp(part_full + 8u * b, (vrow >> 1) & 1u, abort_flag);
        float pr = 0.f;
        if (lane < kSWarps) pr = misc->part[b][lane];
        __syncwarp();
        if (lane == 0 && have) mbar_arrive(part_empty + 8u * b);
        ScaleCoef coef;
        coef.f = 0.f; coef.fix = 0.f; coef.c2 = 0.f; coef.sgn = 0.f; coef.mode = 0;
        if (have) {
          const double S = warp_sum((double)pr);
          bool fallback = !(S > 0.0) || !(S <= kMaxSafeSum) || !isfinite(z_a);
          double lse = (double)z_a + log(S);
          if (fallback) lse = warp_row_lse<InT>(zrow, p.V);
          if (!isfinite(lse)) {
            flags |= DPPO_STATUS_NONFINITE_ROW;
          } else {
            double pi_a;
            int f2 = 0;
            auto pick = [&](const auto* v, int i) { return i == 0 ? v[0] : (i == 1 ? v[1] : (i == 2 ? v[2] : v[3])); };
            auto z_at = [&](int id, int k) {
              if (id == a) return z_a;
              if (k >= 0 && k < 32 * kPre) return pick(zk_pre, k >> 5);
              return to_f32<InT>(zrow[id]);
            };
            auto list_at = [&](int k, int& id, float& pm) {
              if (k < 32 * kPre) { id = pick(id_pre, k >> 5); pm = pick(pm_pre, k >> 5); }
              else { id = p.topk_ids[t * (int64_t)p.K + k]; pm = p.topk_p[t * (int64_t)p.K + k]; }
            };
            row_scalars_warp(p, t, a, lse, scale, z_at, list_at, D, M, g, r, absdiff, pi_a, f2);
            if (f2) { flags |= f2; D = 0.f; M = 0; g = 0.0; r = 0.f; absdiff = 0.f; }
            else if (g != 0.0) {
              const RowCoef rc = make_coef(g, lse, pi_a);
              coef.fix = rc.fix; coef.c2 = rc.c2; coef.sgn = rc.sgn;
              if (fallback) { coef.mode = 2; }
              else { coef.mode = 1; coef.f = (float)(g / S); }
            }
          }
        }
        if (lane == 0) {
          bool ok = have;
          if (ok && vrow >= 2) ok = mbar_wait(coef_empty + 8u * b, ((vrow >> 1) & 1u) ^ 1u, abort_flag);
          if (ok) {
            misc->coef[b] = coef;
            mbar_arrive(coef_full + 8u * b);
          }
        }
        ++vrow;
      }
      if (lane == 0) {
        p.divergence[t] = D;
        p.mask[t] = (uint8_t)M;
        p.row_loss[t] = (float)(-g);
        p.row_r[t] = r;
        p.row_absdiff[t] = absdiff;
        if (flags) atomicOr(p.status, flags);
      }
      meta = meta_next;
    }
  }

  __syncwarp();
  if (*abort_flag) {
    if (lane == 0) atomicOr(p.status, DPPO_STATUS_WAIT_LIMIT);
    // leave time for bulk copies that may still be in flight towards this CTA's shared memory
    const unsigned long long t_exit = globaltimer_ns();
    while (globaltimer_ns() - t_exit < 1000000ull) __nanosleep(1000);
  }
}

// Tuning of the one-exponential kernel (process-wide): slots of the first sweep's ring (the rest feeds the second sweep)
// and how many chunks beyond one row the first sweep may run ahead of the second.  0 = built-in defaults.
std::atomic<int> g_sum_slots{0}, g_lead_extra{0};

int scale_slots(int dev) {
  int max_smem = 0;
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  int n = (max_smem - kSMisc) / kSChunk;
  return n > kSMaxSlots ? kSMaxSlots : n;
}

template <typename InT, typename OutT>
cudaError_t launch_scale_t(const RowParams& p, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int nslots = scale_slots(dev);
  if (nslots < 2) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)nslots * kSChunk + kSMisc;
  cudaError_t e = cudaFuncSetAttribute(dppo_row_scale_kernel<InT, OutT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = (int)(p.T < sms ? p.T : sms);
  dppo_row_scale_kernel<InT, OutT><<<grid, kSThreads, smem, st>>>(p, nslots, g_sum_slots.load(), g_lead_extra.load());
  return cudaGetLastError();
}

}  // namespace

// Rows that start on 16-byte boundaries and are whole 16-byte vectors long, and a gradient tensor that does not overlap
// the logits (the first sweep already writes into it).
bool scale_layout_ok(const RowParams& p, int in_dtype, int out_dtype) {
  const int64_t in_sz = (in_dtype == DPPO_BF16) ? 2 : 4, out_sz = (out_dtype == DPPO_BF16) ? 2 : 4;
  if (in_dtype == DPPO_F32 && out_dtype != DPPO_F32) return false;
  if ((p.V * in_sz) % 16 != 0 || p.V * in_sz >= ((int64_t)1 << 31)) return false;
  if (((uintptr_t)p.logits) % 16 != 0 || (p.ld_in * in_sz) % 16 != 0) return false;
  if (((uintptr_t)p.dlogits) % 16 != 0 || (p.ld_out * out_sz) % 16 != 0) return false;
  if (p.T > 0) {
    const uintptr_t a0 = (uintptr_t)p.logits, a1 = a0 + (uintptr_t)((p.T - 1) * p.ld_in + p.V) * in_sz;
    const uintptr_t b0 = (uintptr_t)p.dlogits, b1 = b0 + (uintptr_t)((p.T - 1) * p.ld_out + p.V) * out_sz;
    if (a0 < b1 && b0 < a1) return false;
  }
  return true;
}

cudaError_t launch_scale(const RowParams& p, int in_dtype, int out_dtype, cudaStream_t st) {
  if (p.T == 0) return cudaSuccess;
  if (in_dtype == DPPO_F32 && out_dtype == DPPO_F32) return launch_scale_t<float, float>(p, st);
  if (in_dtype == DPPO_BF16 && out_dtype == DPPO_BF16) return launch_scale_t<__nv_bfloat16, __nv_bfloat16>(p, st);
  if (in_dtype == DPPO_BF16 && out_dtype == DPPO_F32) return launch_scale_t<__nv_bfloat16, float>(p, st);
  return cudaErrorInvalidValue;
}

}  // namespace dppo

extern "C" void dppo_scale_kernel_tuning(int sum_slots, int lead_chunks_beyond_row) {
  dppo::g_sum_slots.store(sum_slots);
  dppo::g_lead_extra.store(lead_chunks_beyond_row);
}
