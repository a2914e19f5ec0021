// Row kernel for 16-byte aligned layouts: one persistent CTA per SM walks the token rows
// blockIdx.x, blockIdx.x + gridDim.x, ... with two independent streams of bulk asynchronous copies
// (TMA, cp.async.bulk) through two rings of shared-memory slots, connected only by mbarriers:
//
//   sum stream    producer warp S copies the chunks of row n+k from global memory (first touch: HBM,
//                 L2 evict-last hint); 8 sum warps add up exp(z - ref) against a per-thread reference
//                 (moved up only if a chunk would overflow) and hand per-warp partials to a scalar warp
//   scalar warps  (two, taking the rows in turn) log-sum-exp, ratio, divergence, mask, loss term of the
//                 row; post the gradient coefficients
//   grad stream   producer warp G copies the chunks of row n a second time (they were read a few
//                 microseconds earlier by the sum stream and normally still sit in L2; evict-first
//                 hint); 8 grad warps write the gradient with 128-bit streaming stores
//
// Neither stream has to keep a row resident in shared memory, so both run as plain pipelines with
// several chunks in flight; the sum stream leads the grad stream by at most about two rows
// (depth of the coefficient hand-off), which bounds the L2 footprint of rows waiting for their
// second read to roughly 2 x 148 rows.  HBM traffic stays one read and one write of the tensor as
// long as those rows survive in L2.
//
// Every wait is bounded: a wait that runs out sets a shared abort flag and the status bit
// DPPO_STATUS_WAIT_LIMIT; from then on every warp skips its remaining work and returns.
#include <type_traits>

#include "dppo_common.cuh"
#include "dppo_pipe.cuh"
#include "dppo_rowtools.cuh"

namespace dppo {

constexpr int kChunkBytes = 16384;
constexpr int kGroupThreads = 256;              // threads of the sum group and of the grad group
constexpr int kGroupWarps = kGroupThreads / 32;
constexpr int kVecPerThread = kChunkBytes / 16 / kGroupThreads;   // 16-byte vectors per thread per chunk
constexpr int kScalarWarps = 2;     // they take the CTA's valid rows in turn (three would put the CTA at 21 warps, which the
                                    // register file holds only with spills: measured slower)
constexpr int kHand = 2;            // hand-off buffers sum -> scalar -> grad: valid row n uses buffer n % kHand (4 measured the same)
constexpr int kRingThreads = 2 * kGroupThreads + 32 * kScalarWarps + 64;   // + scalar warps + two producer warps
static_assert(kHand >= kScalarWarps, "a buffer per scalar warp at least");
// buffer of valid row n, parity of the barrier phase of that use, and whether the buffer has been used before
struct Hand { uint32_t b, par; bool again; };
__device__ __forceinline__ Hand hand_of(uint32_t n) {
  const uint32_t u = n / (uint32_t)kHand;
  return Hand{n - u * (uint32_t)kHand, u & 1u, n >= (uint32_t)kHand};
}
constexpr int kMiscBytes = 1024;                // barriers + hand-off buffers
constexpr int kMaxSlots = 14;                   // both rings together
constexpr int kMaxCluster = 4;                  // CTAs that may share a row
static_assert(kVecPerThread * kGroupThreads * 16 == kChunkBytes, "chunk geometry");

struct RingMisc {
  unsigned long long full[kMaxSlots];    // chunk landed            (producer -> consumers of that ring)
  unsigned long long empty[kMaxSlots];   // chunk consumed          (consumers -> producer)
  unsigned long long part_full[kHand];       // partials of a row ready (sum -> scalar)
  unsigned long long part_empty[kHand];
  unsigned long long coef_full[kHand];       // coefficients of a row ready (scalar -> grad)
  unsigned long long coef_empty[kHand];
  float2 part[kHand][kGroupWarps];           // (reference, sum of exp) per sum warp
  unsigned long long x_full[kHand];          // clusters: the row's partial of every CTA has arrived (scalar warps -> scalar warp)
  unsigned long long x_empty[kHand];         //           and has been read by every CTA
  float2 x_part[kHand][kMaxCluster];         //           (reference, sum of exp) per CTA of the cluster
  RowCoef coef[kHand];
  int abort_flag;
  unsigned int grad_chunks;              // chunks the grad warps have finished (written by one lane)
};
static_assert(sizeof(RingMisc) <= kMiscBytes, "misc area");

// Where a row lies in the image the ring holds of it.  SH = false: rows start on 16-byte boundaries and their byte
// length is a multiple of 16, the image is the row.  SH = true ("shifted" rows: row starts that are only element
// aligned): the image starts at the 16-byte boundary below the row's first element, `head` bytes early, and the bulk
// copies cover it up to the last boundary inside the row; the few bytes after that are fetched with plain loads.
struct RowGeom {
  uint32_t head;      // bytes in front of the row's first element
  uint32_t xend;      // head + bytes of the row
  uint32_t xa;        // bytes of the image that bulk copies deliver (xend rounded down to 16)
  int C;              // chunks
};
template <typename InT, bool SH>
__device__ __forceinline__ RowGeom row_geom(const RowParams& p, int64_t t, uint32_t row_bytes, int C_static) {
  RowGeom g;
  if (!SH) { g.head = 0; g.xend = row_bytes; g.xa = row_bytes; g.C = C_static; return g; }
  const uintptr_t addr = reinterpret_cast<uintptr_t>(p.logits) + (uintptr_t)(t * p.ld_in) * sizeof(InT);
  g.head = (uint32_t)(addr & 15u);
  g.xend = g.head + row_bytes;
  g.xa = g.xend & ~15u;
  g.C = (int)((g.xend + kChunkBytes - 1) / kChunkBytes);
  return g;
}

// One producer lane: copies every chunk of every valid row of this CTA into the ring
// [first_slot, first_slot + nslots), in order, as slots are released.
template <typename InT, bool SH>
__device__ __forceinline__ void produce_stream(const RowParams& p, uint32_t slots_base, unsigned char* slots_ptr, uint32_t full_base,
                                               uint32_t empty_base, int first_slot, int nslots, uint32_t row_bytes, int C, uint64_t policy,
                                               const WaitCtl& wc, volatile unsigned int* follow, unsigned int lead, int rank, int CL) {
  const char* logits = reinterpret_cast<const char*>(p.logits);
  const int64_t t0 = blockIdx.x / CL, G = gridDim.x / CL;
  RingPos pos{0, 0};
  bool first_lap = true;
  unsigned int issued = 0;
  int meta = load_meta(p, t0);
  for (int64_t t = t0; t < p.T; t += G) {
    const int meta_next = load_meta(p, t + G);
    if (meta >= 0) {
      const RowGeom gm = row_geom<InT, SH>(p, t, row_bytes, C);
      const char* row = logits + t * p.ld_in * (int64_t)sizeof(InT) - gm.head;      // start of the image
      for (int c = rank; c < gm.C; c += CL) {
        const int slot = first_slot + pos.slot;
        if (follow) {                      // stay at most `lead` chunks ahead of the stream we feed L2 for
          if (issued - *follow >= lead) {
            const unsigned long long w0 = globaltimer_ns();
            while (issued - *follow >= lead) {
              if (wc.aborted()) return;
              if (globaltimer_ns() - w0 > wc.limit_ns) { wc.abort(); return; }
              __nanosleep(64);
            }
          }
          ++issued;
        }
        // lap u >= 1 of a slot needs its (u-1)-th release: parity (u-1)&1 = phase^1
        if (!first_lap && !mbar_wait(empty_base + 8u * slot, pos.phase ^ 1u, wc)) return;
        const uint32_t off = (uint32_t)c * kChunkBytes;
        const uint32_t bar = full_base + 8u * slot;
        if (!SH) {
          const uint32_t bytes = (row_bytes - off) < (uint32_t)kChunkBytes ? (row_bytes - off) : (uint32_t)kChunkBytes;
          mbar_arrive_expect_tx(bar, bytes);
          bulk_load(slots_base + (uint32_t)slot * kChunkBytes, row + off, bytes, bar, policy);
        } else {
          const uint32_t bytes = off < gm.xa ? ((gm.xa - off) < (uint32_t)kChunkBytes ? (gm.xa - off) : (uint32_t)kChunkBytes) : 0u;
          // the row's last bytes, past the last 16-byte boundary inside it, belong to this chunk when that boundary
          // does: plain loads (nothing beyond the row is read), stored before the arrival that publishes the chunk
          if (gm.xend > gm.xa && gm.xa >= off && gm.xa < off + (uint32_t)kChunkBytes) {
            const InT* src = reinterpret_cast<const InT*>(row + gm.xa);
            InT* dst = reinterpret_cast<InT*>(slots_ptr + (size_t)slot * kChunkBytes + (gm.xa - off));
            for (uint32_t i = 0; i < (gm.xend - gm.xa) / (uint32_t)sizeof(InT); ++i) dst[i] = src[i];
          }
          if (bytes) {
            mbar_arrive_expect_tx(bar, bytes);
            bulk_load(slots_base + (uint32_t)slot * kChunkBytes, row + off, bytes, bar, policy);
          } else {
            mbar_arrive(bar);
          }
        }
        if (++pos.slot == nslots) { pos.slot = 0; pos.phase ^= 1u; first_lap = false; }
      }
    }
    meta = meta_next;
  }
}

// Element-wise store of the valid part of a vector at the edge of a shifted row: element i of the vector sits at byte
// xo + i * sizeof(OutT) of the row's image and is written iff that lies in [head, xend).
template <typename OutT, int N>
__device__ __forceinline__ void store_edge(OutT* row_image, uint32_t xo, const float* v, uint32_t sign2, uint32_t head, uint32_t xend) {
#pragma unroll
  for (int i = 0; i < N; ++i) {
    const uint32_t pos = xo + (uint32_t)i * (uint32_t)sizeof(OutT);
    if (pos >= head && pos < xend) row_image[pos / (uint32_t)sizeof(OutT)] = from_f32<OutT>(sign2 ? -v[i] : v[i]);
  }
}

// CL > 1: launched as clusters of CL CTAs that share each row (CTA r takes the chunks r, r + CL, ...): long rows, of which
// one per CTA would not fit L2 between their two reads.  The sum warps hand their partials to the scalar warps of all CL
// CTAs, every CTA works out the row's scalars for its own gradient warps, and the first one writes the row's outputs.
template <typename InT, typename OutT, bool SH, int CL>
__global__ void __launch_bounds__(kRingThreads, 1) dppo_row_ring_kernel(RowParams p, int nslots) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int N = Vec<InT>::N;
  RingMisc* misc = reinterpret_cast<RingMisc*>(smem + (size_t)nslots * kChunkBytes);
  const uint32_t slots_base = smem_u32(smem);
  const uint32_t full_base = smem_u32(&misc->full[0]);
  const uint32_t empty_base = smem_u32(&misc->empty[0]);
  const uint32_t part_full = smem_u32(&misc->part_full[0]), part_empty = smem_u32(&misc->part_empty[0]);
  const uint32_t coef_full = smem_u32(&misc->coef_full[0]), coef_empty = smem_u32(&misc->coef_empty[0]);
  const WaitCtl wc{&misc->abort_flag, p.wait_ns};
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rank = (CL > 1) ? (int)cluster_ctarank() : 0;
  // slots [0, ns_sum) feed the sum warps, [ns_sum, nslots) the grad warps; the second read comes from L2 with a
  // shorter latency but is issued as early as possible, so the grad ring gets the larger share (4 + 10 of 14)
  const int ns_sum = (2 * nslots + 3) / 7 < 2 ? 2 : (2 * nslots + 3) / 7, ns_grad = nslots - ns_sum;

  if (tid == 0) {
    for (int i = 0; i < nslots; ++i) {
      mbar_init(full_base + 8u * i, 1);
      mbar_init(empty_base + 8u * i, kGroupWarps);
    }
    for (int i = 0; i < kHand; ++i) {
      mbar_init(part_full + 8u * i, kGroupWarps);
      mbar_init(part_empty + 8u * i, 1);
      mbar_init(smem_u32(&misc->x_full[i]), CL);
      mbar_init(smem_u32(&misc->x_empty[i]), CL);
      mbar_init(coef_full + 8u * i, 1);
      mbar_init(coef_empty + 8u * i, kGroupWarps);
    }
    misc->abort_flag = 0;
    misc->grad_chunks = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (CL > 1) cluster_sync_all();       // the peers' barriers exist before anything is sent to them

  const uint32_t row_bytes = (uint32_t)(p.V * (int64_t)sizeof(InT));     // launcher guarantees < 2^31
  const int C = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);      // chunks per row (shifted rows: of most rows)
  const int64_t t0 = blockIdx.x / CL, G = gridDim.x / CL;      // rows t0, t0 + G, ... of this CTA (of its cluster)
  const int C_own = (C + CL - 1) / CL;                          // chunks of a row this CTA streams (at most)

  if (warp >= 2 * kGroupWarps + kScalarWarps) {
    // ------------------------------------------------------------------ producers (one lane each)
    // (test injection: the producers issue nothing, so that every consumer wait of the CTA runs out)
    if (lane == 0 && !(p.inject & DPPO_INJECT_NO_COPIES)) {
      uint64_t policy;
      if (warp == 2 * kGroupWarps + kScalarWarps) {
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
        // The sum stream runs at most one row and a few chunks ahead of the grad warps (at least one row, or
        // the grad warps could never get their coefficients).  Rows between their first and second read then
        // occupy about #SMs x lead chunks of L2 (71 MB at V = 151936 bf16); a longer lead makes the second
        // read miss L2, a shorter one leaves the sum warps idle, and the chunks beyond the row are also the time
        // the scalar warp has for a row (its stage is longest for the Top-K variants: with C + 7 they ran 3 - 8 %
        // slower than the Binary ones, from C + 11 on all variants run alike).  Measured on B200: C + 11 .. C + 15.
        const int lead = (C_own + 11 <= 30) ? C_own + 11 : ((C_own + 2 > 30) ? C_own + 2 : 30);
        produce_stream<InT, SH>(p, slots_base, smem, full_base, empty_base, 0, ns_sum, row_bytes, C, policy, wc,
                                &misc->grad_chunks, (unsigned int)lead, rank, CL);
      } else {
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        produce_stream<InT, SH>(p, slots_base, smem, full_base, empty_base, ns_sum, ns_grad, row_bytes, C, policy, wc, nullptr, 0u, rank, CL);
      }
    }
  } else if (warp < kGroupWarps) {
    // ------------------------------------------------------------------ sum warps: sweep 1
    const uint32_t gtid = (uint32_t)tid;
    RingPos pos{0, 0};
    uint32_t vrow = 0;
    int meta = load_meta(p, t0);
    for (int64_t t = t0; t < p.T; t += G) {
      const int meta_next = load_meta(p, t + G);
      if (__shfl_sync(0xffffffffu, (int)wc.aborted(), 0)) break;
      if (meta >= 0) {
        // per-thread partial: s = sum exp(z - ref); ref is the maximum of the thread's first entries
        // and moves up only when a chunk's sum shows that an entry exceeds it by > 44
        // the sampled token's entry is left out of the sums (the scalar warp adds it: 1 - pi(a) then comes from the
        // sum over the other entries and keeps its relative accuracy when pi(a) is close to 1); see below how
        float ref = -INFINITY, nm = 0.f, s = 0.f;
        const RowGeom gm = row_geom<InT, SH>(p, t, row_bytes, C);
        constexpr uint32_t kChunkElems = kChunkBytes / sizeof(InT);
        const uint32_t a_img = (uint32_t)meta + gm.head / (uint32_t)sizeof(InT);   // the sampled token's place in the image,
        const int a_chunk = (int)(a_img / kChunkElems);                            // the chunk that holds it
        const uint32_t a_loc = a_img % kChunkElems;                                // and its place in that chunk
        for (int c = rank; c < gm.C; c += CL) {
          const bool ok = mbar_wait_warp(full_base + 8u * pos.slot, pos.phase, wc);
          const uint32_t cbase = (uint32_t)c * kChunkBytes;
          const uint32_t sbase = slots_base + (uint32_t)pos.slot * kChunkBytes;
          const bool has_a = (c == a_chunk);                                       // warp-uniform
          if (ok) {
            // The sampled token's entry is taken out of the sums by overwriting it with -inf in the slot, by the one
            // thread that reads its vector (program order makes the store visible to that thread's own loads, no other
            // thread reads that vector, and the gradient sweep reads the row from its own ring).  Selecting the entry in
            // registers instead costs the straight-line path 2 - 3 % although it runs once per row.  The fence orders
            // this generic-proxy write before the bulk copy that refills the slot later.
            if (has_a && (a_loc / N) % kGroupThreads == gtid) {
              if (sizeof(InT) == 2) asm volatile("st.shared.b16 [%0], %1;" ::"r"(sbase + a_loc * 2u), "h"((unsigned short)0xFF80) : "memory");
              else asm volatile("st.shared.b32 [%0], %1;" ::"r"(sbase + a_loc * 4u), "r"(0xFF800000u) : "memory");
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            // chunks that the bulk copy filled completely take the straight-line path
            const bool full_chunk = cbase + (uint32_t)kChunkBytes <= gm.xa;
            bool done = false;
            // straight-line path: all loads first, then 4 x N independent exponentials.  TAIL: the row's last chunk when
            // the row ends on a 16-byte boundary: vectors beyond the row are replaced by -inf (probability zero)
            auto straight = [&](auto tail_c) {
              constexpr bool TAIL = decltype(tail_c)::value;
              uint4 v[kVecPerThread];
#pragma unroll
              for (int k = 0; k < kVecPerThread; ++k) v[k] = lds128(sbase + ((uint32_t)k * kGroupThreads + gtid) * 16u);
              if (TAIL) {
                constexpr uint32_t ninf = sizeof(InT) == 2 ? 0xFF80FF80u : 0xFF800000u;
#pragma unroll
                for (int k = 0; k < kVecPerThread; ++k)
                  if (cbase + ((uint32_t)k * kGroupThreads + gtid) * 16u >= gm.xa) v[k] = make_uint4(ninf, ninf, ninf, ninf);
              }
              float z[kVecPerThread][N];
#pragma unroll
              for (int k = 0; k < kVecPerThread; ++k) Vec<InT>::unpack(v[k], z[k]);
              if (SH && c == 0 && gtid == 0) {    // a shifted row's image starts with entries that are not the row's
#pragma unroll
                for (int i = 0; i < N; ++i)
                  if ((uint32_t)i * (uint32_t)sizeof(InT) < gm.head) z[0][i] = -INFINITY;
              }
              if (ref == -INFINITY) {            // first chunk of the row: reference = maximum of the thread's first vector
                float vm = z[0][0];              // (any finite entry would do: a chunk whose sum overflows moves it up)
#pragma unroll
                for (int i = 1; i < N; ++i) vm = fmaxf(vm, z[0][i]);
                if (vm != -INFINITY) { ref = vm; nm = -vm * kLog2e; }
              }
              // exponent arguments and partial sums on pairs of fp32 lanes (one instruction per two elements)
              const float2 l2 = make_float2(kLog2e, kLog2e), nm2 = make_float2(nm, nm);
              float2 acc2[kVecPerThread];
#pragma unroll
              for (int k = 0; k < kVecPerThread; ++k) {
                float2 e2[N / 2];
#pragma unroll
                for (int i = 0; i < N / 2; ++i) {
                  const float2 arg = __ffma2_rn(make_float2(z[k][2 * i], z[k][2 * i + 1]), l2, nm2);
                  e2[i] = make_float2(ex2_approx(arg.x), ex2_approx(arg.y));
                }
#pragma unroll
                for (int w = 1; w < N / 2; w <<= 1)
#pragma unroll
                  for (int i = 0; i + w < N / 2; i += 2 * w) e2[i] = __fadd2_rn(e2[i], e2[i + w]);
                acc2[k] = e2[0];
              }
#pragma unroll
              for (int w = 1; w < kVecPerThread; w <<= 1)
#pragma unroll
                for (int k = 0; k + w < kVecPerThread; k += 2 * w) acc2[k] = __fadd2_rn(acc2[k], acc2[k + w]);
              const float acc = acc2[0].x + acc2[0].y;
              if (acc <= 7.3786976e19f && ref != -INFINITY) { s += acc; done = true; }   // <= 2^66, not NaN
            };
            if (full_chunk) straight(std::false_type{});
            else if (!SH) straight(std::true_type{});
            if (!done) {
              // tail chunk, or an entry far above the reference (or NaN): vector by vector, moving the reference up
#pragma unroll 1
              for (int k = 0; k < kVecPerThread; ++k) {
                const uint32_t off = ((uint32_t)k * kGroupThreads + gtid) * 16u;
                if (cbase + off < gm.xend) {
                  const uint4 v = lds128(sbase + off);
                  float z[N];
                  Vec<InT>::unpack(v, z);
                  if (SH) {                         // entries of the image outside the row count as probability zero
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                      const uint32_t pos_b = cbase + off + (uint32_t)i * (uint32_t)sizeof(InT);
                      if (pos_b < gm.head || pos_b >= gm.xend) z[i] = -INFINITY;
                    }
                  }
                  float vm = z[0];
#pragma unroll
                  for (int i = 1; i < N; ++i) vm = fmaxf(vm, z[i]);
                  if (vm > ref) {
                    s *= ex2_approx((ref - vm) * kLog2e);     // ref = -inf gives 0 * 0
                    ref = vm;
                    nm = -vm * kLog2e;
                  }
                  if (ref != -INFINITY) {
                    float vs = 0.f;
#pragma unroll
                    for (int i = 0; i < N; ++i) vs += ex2_approx(fmaf(z[i], kLog2e, nm));
                    s += vs;
                  }
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_base + 8u * pos.slot);
          pos.advance(ns_sum);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float m2 = __shfl_xor_sync(0xffffffffu, ref, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
          merge_ms(ref, s, m2, s2);
        }
        if (lane == 0) {
          const Hand h = hand_of(vrow);
          const uint32_t b = h.b;
          bool ok = true;
          if (h.again) ok = mbar_wait(part_empty + 8u * b, h.par ^ 1u, wc);
          if (ok) {
            misc->part[b][warp] = make_float2(ref, s);
            mbar_arrive(part_full + 8u * b);
          }
        }
        ++vrow;
      }
      meta = meta_next;
    }
  } else if (warp < 2 * kGroupWarps) {
    // ------------------------------------------------------------------ grad warps: sweep 2
    const uint32_t gtid = (uint32_t)(tid - kGroupThreads);
    OutT* dlogits = reinterpret_cast<OutT*>(p.dlogits);
    RingPos pos{0, 0};
    uint32_t vrow = 0;
    unsigned int chunks_done = 0;
    int meta = load_meta(p, t0);
    for (int64_t t = t0; t < p.T; t += G) {
      const int meta_next = load_meta(p, t + G);
      if (__shfl_sync(0xffffffffu, (int)wc.aborted(), 0)) break;
      OutT* drow = dlogits + t * p.ld_out;
      const RowGeom gm = row_geom<InT, SH>(p, t, row_bytes, C);
      // shifted rows: the output row is shifted by the same number of bytes (same element size, same misalignment, the
      // launcher checks), so whole vectors of the image are whole, aligned vectors of the output
      if (SH) drow = reinterpret_cast<OutT*>(reinterpret_cast<char*>(drow) - gm.head);
      const uint32_t head_e = gm.head / (uint32_t)sizeof(InT);         // elements of the image in front of the row
      if (meta < 0) {
        const float zero[N] = {};
        const uint32_t zt = (uint32_t)rank * kGroupThreads + gtid, zn = (uint32_t)CL * kGroupThreads;   // among the CTAs that share the row
        if (!SH) {
          for (uint32_t j0 = zt * N; j0 < (uint32_t)p.V; j0 += zn * N) Store<OutT, N>::run(drow, j0, zero);
        } else {
          for (uint32_t xo = zt * 16u; xo < gm.xend; xo += zn * 16u) {
            if (xo >= gm.head && xo + 16u <= gm.xend) Store<OutT, N>::run(drow, xo / (uint32_t)sizeof(InT), zero);
            else store_edge<OutT, N>(drow, xo, zero, 0u, gm.head, gm.xend);
          }
        }
      } else {
        const Hand h = hand_of(vrow);
        const uint32_t b = h.b;
        const bool have = mbar_wait_warp(coef_full + 8u * b, h.par, wc);
        RowCoef coef = misc->coef[b];
        __syncwarp();
        if (lane == 0 && have) mbar_arrive(coef_empty + 8u * b);
        if (!have) coef.zero_row = 1;
        const uint32_t sign2 = (coef.sgn < 0.f) ? 0x80008000u : 0u;
        const uint32_t a = (uint32_t)meta + head_e;                    // the sampled token's place in the image
        for (int c = rank; c < gm.C; c += CL) {
          const int slot = ns_sum + pos.slot;
          const bool ok = mbar_wait_warp(full_base + 8u * slot, pos.phase, wc);
          const uint32_t cbase = (uint32_t)c * kChunkBytes;
          const uint32_t sbase = slots_base + (uint32_t)slot * kChunkBytes;
          if (ok) {
            const bool full_chunk = cbase + (uint32_t)kChunkBytes <= gm.xa;
            const uint32_t e0 = cbase / (uint32_t)sizeof(InT);                       // first element of the chunk
            const bool has_a = (a - e0) < (uint32_t)(kChunkBytes / sizeof(InT));     // warp-uniform
            // straight-line path: all loads first, 4 x N independent exponentials, 4 stores.  TAIL: the row's last chunk
            // when the row ends on a 16-byte boundary: vectors beyond the row are not stored
            auto straight = [&](auto tail_c) {
              constexpr bool TAIL = decltype(tail_c)::value;
              uint4 raw[kVecPerThread];
#pragma unroll
              for (int k = 0; k < kVecPerThread; ++k) raw[k] = lds128(sbase + ((uint32_t)k * kGroupThreads + gtid) * 16u);
#pragma unroll
              for (int k = 0; k < kVecPerThread; ++k) {
                float z[N], v[N];
                Vec<InT>::unpack(raw[k], z);
                const float2 l2 = make_float2(kLog2e, kLog2e), c22 = make_float2(coef.c2, coef.c2);
#pragma unroll
                for (int i = 0; i < N; i += 2) {
                  const float2 arg = __ffma2_rn(make_float2(z[i], z[i + 1]), l2, c22);
                  v[i] = ex2_approx(arg.x);
                  v[i + 1] = ex2_approx(arg.y);
                }
                if (SH && c == 0 && k == 0 && gtid == 0 && gm.head != 0) store_edge<OutT, N>(drow, 0u, v, sign2, gm.head, gm.xend);
                else if (!TAIL || cbase + ((uint32_t)k * kGroupThreads + gtid) * 16u < gm.xa)
                  Store<OutT, N>::run(drow, e0 + ((uint32_t)k * kGroupThreads + gtid) * N, v, sign2);
              }
            };
            if (!coef.zero_row && !has_a && (full_chunk || !SH)) {
              if (full_chunk) straight(std::false_type{}); else straight(std::true_type{});
            } else {
#pragma unroll 1
              for (int k = 0; k < kVecPerThread; ++k) {
                const uint32_t off = ((uint32_t)k * kGroupThreads + gtid) * 16u;
                if (cbase + off < gm.xend) {
                  const uint32_t j0 = (cbase + off) / (uint32_t)sizeof(InT);
                  float v[N];
                  if (coef.zero_row) {
#pragma unroll
                    for (int i = 0; i < N; ++i) v[i] = 0.f;
                  } else {
                    const uint4 raw = lds128(sbase + off);
                    float z[N];
                    Vec<InT>::unpack(raw, z);
#pragma unroll
                    for (int i = 0; i < N; ++i) v[i] = ex2_approx(fmaf(z[i], kLog2e, coef.c2));
                    if (a - j0 < (uint32_t)N) {             // the sampled token's entry is g * (pi(a) - 1)
#pragma unroll
                      for (int i = 0; i < N; ++i)
                        if (j0 + i == a) v[i] = coef.fix * coef.sgn;   // the store flips it back
                    }
                  }
                  if (!SH || (cbase + off >= gm.head && cbase + off + 16u <= gm.xend)) Store<OutT, N>::run(drow, j0, v, sign2);
                  else store_edge<OutT, N>(drow, cbase + off, v, sign2, gm.head, gm.xend);
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_base + 8u * slot);
          ++chunks_done;
          if (tid == kGroupThreads) *(volatile unsigned int*)&misc->grad_chunks = chunks_done;
          pos.advance(ns_grad);
        }
        ++vrow;
      }
      meta = meta_next;
    }
  } else {
    // ------------------------------------------------------------------ scalar warps
    // The scalar warps take the CTA's valid rows in turn, so that a row's scalar stage (a dependent global load, fp64
    // exponentials and logarithms, for the Top-K variants a gather of K logits) may take several row times: with short
    // rows (a vocabulary of 32 000 is four chunks) one warp cannot keep up.  Rows without a sweep go to warp 0.
    const uint32_t sw = (uint32_t)(warp - 2 * kGroupWarps);
    const double scale = p.hdr->scale;
    const bool topk = (p.variant == DPPO_TOPK_TV || p.variant == DPPO_TOPK_KL) && p.K > 0;
    uint32_t vrow = 0;
    int meta = load_meta(p, t0);
    for (int64_t t = t0; t < p.T; t += G) {
      const int meta_next = load_meta(p, t + G);
      if (__shfl_sync(0xffffffffu, (int)wc.aborted(), 0)) break;
      if (kScalarWarps > 1 && ((meta >= 0) ? (vrow % (uint32_t)kScalarWarps) : 0u) != sw) {      // another warp's row
        if (meta >= 0) ++vrow;
        meta = meta_next;
        continue;
      }
      int flags = (meta == -2) ? DPPO_STATUS_BAD_SAMPLED_ID : 0;
      float D = 0.f, r = 0.f, absdiff = 0.f;
      int M = 0;
      double g = 0.0;
      if (meta >= 0) {
        const int a = meta;
        const Hand h = hand_of(vrow);
        const uint32_t b = h.b;
        const InT* zrow = reinterpret_cast<const InT*>(p.logits) + t * p.ld_in;
        const float z_a = to_f32<InT>(zrow[a]);                       // in flight while we wait for the partials
        // Top-K variants: this lane's list entries (positions lane, lane + 32, ...) and their logits are fetched now
        // too, so that the two dependent memory latencies (id, then z[id]) do not sit between the row's sums and
        // its gradient; positions beyond 32 * kPre are loaded when the scalar stage asks for them
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
        bool have = mbar_wait_warp(part_full + 8u * b, h.par, wc);
        float2 pr = make_float2(-INFINITY, 0.f);
        if (lane < kGroupWarps) pr = misc->part[b][lane];
        __syncwarp();
        if (lane == 0 && have) mbar_arrive(part_empty + 8u * b);
        if (CL > 1) {
          // The CTAs that share the row exchange one partial each, scalar warp to scalar warp (the sum warps never wait
          // for another CTA): this CTA's sum warps' partials are merged into one, lane r sends it to CTA r once every
          // CTA has read the buffer's previous content, and the row goes on when all CL partials are here.
          float cm = pr.x;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
          double cp = 0.0;
          if (pr.y > 0.f || pr.y != pr.y) cp = (double)pr.y * exp((double)pr.x - (double)cm);
          const float cs = (float)warp_sum(cp);
          const uint32_t xf = smem_u32(&misc->x_full[b]), xe = smem_u32(&misc->x_empty[b]);
          if (have && h.again) have = __all_sync(0xffffffffu, mbar_wait_cluster(xe, h.par ^ 1u, wc));
          if (have && lane < CL) {
            st_cluster_f32x2(map_to_cta(smem_u32(&misc->x_part[b][rank]), (uint32_t)lane), cm, cs);
            bar_arrive_cluster(map_to_cta(xf, (uint32_t)lane));
          }
          if (have) have = __all_sync(0xffffffffu, mbar_wait_cluster(xf, h.par, wc));
          pr = make_float2(-INFINITY, 0.f);
          if (have && lane < CL) pr = misc->x_part[b][lane];
          __syncwarp();
          if (have && lane < CL) bar_arrive_cluster(map_to_cta(xe, (uint32_t)lane));
        }
        RowCoef coef;
        coef.c2 = 0.f; coef.sgn = 0.f; coef.fix = 0.f; coef.zero_row = 1;
        if (have) {
          float mm = pr.x;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
          double part = 0.0;
          if (pr.y > 0.f || pr.y != pr.y) part = (double)pr.y * exp((double)pr.x - (double)mm);
          const double S_o = warp_sum(part);                 // sum over the entries other than the sampled token
          double lse, log_other;
          combine_lse((double)mm, S_o, (double)z_a, lse, log_other);
          if (!isfinite(lse)) {
            flags |= DPPO_STATUS_NONFINITE_ROW;
          } else {
            double pi_a;
            int f2 = 0;
            // this lane only ever asks for its own list positions k = lane + 32 i
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
            row_scalars_warp(p, t, a, lse, log_other, scale, z_at, list_at, D, M, g, r, absdiff, pi_a, f2);
            if (f2) { flags |= f2; D = 0.f; M = 0; g = 0.0; r = 0.f; absdiff = 0.f; }
            else coef = make_coef(g, lse, pi_a);
          }
        }
        if (lane == 0) {
          bool ok = have;
          if (ok && h.again) ok = mbar_wait(coef_empty + 8u * b, h.par ^ 1u, wc);
          if (ok) {
            misc->coef[b] = coef;
            mbar_arrive(coef_full + 8u * b);
          }
        }
        ++vrow;
      }
      if (lane == 0 && rank == 0) {
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
  if (wc.aborted()) {
    if (lane == 0) atomicOr(p.status, DPPO_STATUS_WAIT_LIMIT);
    drain_after_abort();
  }
  // the CTAs of a cluster leave together: a peer may still be sending partials or arrivals to this one's shared memory
  if (CL > 1) cluster_sync_all();
}

static int ring_slots(int dev) {
  int max_smem = 0;
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  int n = (max_smem - kMiscBytes) / kChunkBytes;
  return n > kMaxSlots ? kMaxSlots : n;
}

// 1: rows start on 16-byte boundaries and are whole 16-byte vectors long; 2: "shifted" rows (16-byte aligned tensors of
// equal element size whose rows start at the same offset from a 16-byte boundary in logits and dlogits, e.g. contiguous
// tensors with a vocabulary that is not a multiple of 8); 0: neither, the generic kernel takes the call.
static int ring_mode(const RowParams& p, int in_dtype, int out_dtype) {
  const int64_t in_sz = (in_dtype == DPPO_BF16) ? 2 : 4, out_sz = (out_dtype == DPPO_BF16) ? 2 : 4;
  if (in_dtype == DPPO_F32 && out_dtype != DPPO_F32) return 0;
  if (p.V * in_sz + 16 >= ((int64_t)1 << 31)) return 0;
  if (((uintptr_t)p.logits) % 16 != 0 || ((uintptr_t)p.dlogits) % 16 != 0) return 0;
  if ((p.V * in_sz) % 16 == 0 && (p.ld_in * in_sz) % 16 == 0 && (p.ld_out * out_sz) % 16 == 0) return 1;
  if (in_sz == out_sz && (p.ld_in * in_sz) % 16 == (p.ld_out * out_sz) % 16) return 2;
  return 0;
}

bool ring_layout_ok(const RowParams& p, int in_dtype, int out_dtype) { return ring_mode(p, in_dtype, out_dtype) != 0; }

// CTAs that share a row.  One CTA per row needs a lead of one row plus a margin (11 chunks) within the 30 chunks per CTA
// that L2 holds between the two reads (a higher cap was measured slower): rows of up to 19 chunks have it in full, and
// from 21 chunks on two CTAs per row are faster, four for rows of more than 64 chunks (a device of 148 SMs runs only 33
// clusters of four at a time).  Measured on B200, bf16, fraction of the HBM copy peak with 1 / 2 CTAs per row: 19 chunks
// (V = 155 648) 0.87 / 0.82; 22 chunks 0.80 / 0.84; 24 chunks 0.79 / 0.82; 27 chunks 0.79 / 0.82; 32 chunks 0.74 / 0.81
// (four: 0.77); 128 chunks (V = 2^20) 0.66 / 0.66 (four: 0.69).
static int ring_cluster(int64_t row_bytes) {
  const int64_t C = (row_bytes + kChunkBytes - 1) / kChunkBytes;
  return C <= 20 ? 1 : (C <= 64 ? 2 : kMaxCluster);
}

template <typename InT, typename OutT, bool SH, int CL>
static cudaError_t launch_ring_c(const RowParams& p, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int nslots = ring_slots(dev);
  if (nslots < 2) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)nslots * kChunkBytes + kMiscBytes;
  auto kernel = dppo_row_ring_kernel<InT, OutT, SH, CL>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (CL == 1) {
    const int grid = (int)(p.T < sms ? p.T : sms);
    kernel<<<grid, kRingThreads, smem, st>>>(p, nslots);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CL; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(kRingThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // one cluster per set of CL SMs that the device can run at a time (the kernel is persistent: a cluster that had to
  // wait for a free place would run after all others); asked once per device
  static int max_clusters[64] = {};
  int nc = (dev >= 0 && dev < 64) ? max_clusters[dev] : 0;
  if (nc <= 0) {
    cfg.gridDim = dim3((unsigned)(sms / CL * CL), 1, 1);
    e = cudaOccupancyMaxActiveClusters(&nc, kernel, &cfg);
    if (e != cudaSuccess || nc <= 0) {      // no room for such clusters on this device: one CTA per row
      (void)cudaGetLastError();
      return launch_ring_c<InT, OutT, SH, 1>(p, st);
    }
    if (nc > sms / CL) nc = sms / CL;
    if (dev >= 0 && dev < 64) max_clusters[dev] = nc;
  }
  const int64_t clusters = p.T < nc ? p.T : nc;
  cfg.gridDim = dim3((unsigned)(clusters * CL), 1, 1);
  return cudaLaunchKernelEx(&cfg, kernel, p, nslots);
}

template <typename InT, typename OutT, bool SH>
static cudaError_t launch_ring_t(const RowParams& p, cudaStream_t st) {
  switch (p.row_cluster > 0 ? p.row_cluster : ring_cluster(p.V * (int64_t)sizeof(InT))) {
    case 1: return launch_ring_c<InT, OutT, SH, 1>(p, st);
    case 2: return launch_ring_c<InT, OutT, SH, 2>(p, st);
    default: return launch_ring_c<InT, OutT, SH, 4>(p, st);
  }
}

cudaError_t launch_ring(const RowParams& p, int in_dtype, int out_dtype, cudaStream_t st) {
  if (p.T == 0) return cudaSuccess;
  const int mode = ring_mode(p, in_dtype, out_dtype);
  if (mode == 2) {
    if (in_dtype == DPPO_F32 && out_dtype == DPPO_F32) return launch_ring_t<float, float, true>(p, st);
    if (in_dtype == DPPO_BF16 && out_dtype == DPPO_BF16) return launch_ring_t<__nv_bfloat16, __nv_bfloat16, true>(p, st);
    return cudaErrorInvalidValue;
  }
  if (mode != 1) return cudaErrorInvalidValue;
  if (in_dtype == DPPO_F32 && out_dtype == DPPO_F32) return launch_ring_t<float, float, false>(p, st);
  if (in_dtype == DPPO_BF16 && out_dtype == DPPO_BF16) return launch_ring_t<__nv_bfloat16, __nv_bfloat16, false>(p, st);
  if (in_dtype == DPPO_BF16 && out_dtype == DPPO_F32) return launch_ring_t<__nv_bfloat16, float, false>(p, st);
  return cudaErrorInvalidValue;
}

}  // namespace dppo
