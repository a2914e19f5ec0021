// bf16 "TN" GEMM on the 5th-generation tensor cores: C[M,N] = A[M,K] * B[N,K]^T, both operands K-major
// (row-major with K contiguous), fp32 accumulation in tensor memory, epilogue chosen at compile time.
//
// One persistent CTA per SM (192 threads):
//   warp 0      TMA producer: cp.async.bulk.tensor loads of 128x64 (A) and 256x64 (B) bf16 boxes, 128-byte swizzle,
//               into a 4-stage shared-memory ring (mbarrier complete_tx)
//   warp 1      allocates the 512 tensor-memory columns and issues tcgen05.mma (cta_group::1, kind::f16, M=128, N=256,
//               K=16 per instruction); tcgen05.commit releases smem stages and publishes finished accumulators
//   warps 2-5   epilogue: tcgen05.ld of the accumulator (one row per thread, 32 columns at a time) while the MMA warp
//               already fills the other 256-column accumulator buffer
// Tiles are walked M-fastest so that CTAs running at the same time share B strips through L2 (or N-fastest, on request,
// to share A strips).  Epilogues: fp32 store with an optional row factor (or added to the output by L2 reductions; plain
// outputs go through shared memory and bulk tensor stores / reduce-adds);
// exponentials against a per-row reference with their row sums; per-tile softmax statistics with an online maximum;
// finished gradient rows.  With a partial-sum buffer the store variant cuts the tiles of its last, partial wave along K
// (struct Plan) and a second kernel adds the segments up in a fixed order: no atomics, the same bits every time.
// Every mbarrier wait is bounded; on expiry the CTA raises DPPO_STATUS_WAIT_LIMIT, skips the rest and frees its TMEM.
//
// CG = 2 runs the same roles on pairs of CTAs (a cluster of two SMs) with tcgen05.mma.cta_group::2: one work unit is a
// 256 x 256 tile, each CTA stages its own 128 rows of A and only half of the B tile (128 of the 256 columns) and
// accumulates its 128 rows x 256 columns in its own tensor memory; the tensor cores of both SMs read both halves of B.
// That halves the shared-memory fill per flop for B and makes room for 6 stages.  The even CTA of the pair (the leader)
// issues the MMAs; the loads of both CTAs report to the leader's "full" barrier, tcgen05.commit multicasts the "stage
// free" and "accumulator ready" arrivals to both CTAs, and the epilogue warps of both CTAs release the accumulator buffer
// on the leader's barrier.  No multicast loads are used.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dppo.h"
#include "dppo_pipe.cuh"

namespace dppo {
namespace gemm {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr int MAX_STAGES = 6;

// Per-CTA staging for CTA groups of CG = 1 or 2 SMs.
template <int CG> struct Cfg {
  static constexpr int TILE_M = BM * CG;                   // rows of C per work unit (128 per CTA)
  static constexpr int B_COLS = BN / CG;                   // columns of the B tile this CTA stages
  static constexpr int A_STAGE_BYTES = BM * BK * 2, B_STAGE_BYTES = B_COLS * BK * 2;
  static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
  static constexpr int STAGES = (CG == 1) ? 4 : 6;
  // store epilogue through shared memory: two buffers of 32 rows x 32 fp32 columns per epilogue warp
  static constexpr int OUT_BYTES = 4 * 2 * 32 * 32 * 4;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + OUT_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

enum { EPI_STORE_F32 = 0, EPI_STATS = 1, EPI_GRAD = 2, EPI_EXP = 3 };

struct Params {
  int M, N, K;
  // EPI_STORE_F32
  float* C;
  int64_t ldc;
  float* sk_part;        // EPI_STORE_F32 (no transposed store, no accumulation): when the tiles do not fill whole waves of
                         // CTA groups, the tiles of the last, partial wave are cut along K into up to kMaxSegs segments
                         // that are dealt to all groups; their partial tiles land here ([kMaxSegs * groups] slots of
                         // TILE_M x BN floats) and gemm_streamk_fixup_kernel adds them up in a fixed order.  null: whole
                         // tiles only
  // Live extents, read from device memory at kernel start (null: the static M / K).  Rows of A at and beyond *m_live
  // get no output tile (at least one tile is always processed); K blocks at and beyond *k_live are not read (at least
  // one is), so the operands must hold zeros from *k_live to the end of that block.
  const int* m_live;
  const int* k_live;
  const int* row_map;    // EPI_STORE_F32: output row of tile row i (null: i); rows >= *m_live are not stored
  const float* row_scale;  // EPI_STORE_F32: tile row i of the product is multiplied by row_scale[i] (null: 1)
  int c_transposed;      // EPI_STORE_F32 (no K split, no row map): the product is stored transposed, C[col * ldc + row]
  int allow_empty;       // 1: *m_live == 0 means no tile at all (default: one row of tiles is always processed)
  int n_fastest;         // order of the tiles: 0 = M-fastest (CTAs running together share strips of B through L2),
                         // 1 = N-fastest (they share strips of A: for few tiles along N and a large A)
  // EPI_STATS: per (row, n-tile) partial (max, sum exp(z - max)); z at the sampled id
  float2* part;          // [M, tiles_n]
  float* z_a;            // [M]
  const int32_t* ids;    // [M] sampled id per row (EPI_STATS, EPI_GRAD)
  // EPI_GRAD: P[row, col] = sgn * 2^(z*log2e + c2), entry at ids[row] = fix; written as bf16
  const float* c2;       // [M]
  const float* sgn;      // [M] +1, -1, or 0 (zero row)
  const float* fix;      // [M]
  __nv_bfloat16* P;
  int64_t ldp;
  __nv_bfloat16* Pt;     // optional transposed copy [N, ldpt] (same values)
  int64_t ldpt;
  const int* p_row_map;  // EPI_GRAD: row of P that tile row i is written to (null: i; < 0: not written); with a map only
                         // the rows below *m_live are written
  // EPI_EXP: E[row, col] = 2^(z*log2e - cref2[row]) in bf16 (written to P), per (row, n-tile) the fp32 sum of those
  // exponentials before rounding, and z at the sampled id
  const float* cref2;    // [M] per-row reference exponent, log2 units
  float* psum;           // [M, tiles_n]
  const int* e_live;     // rows of E that later steps read: rows below max(64, *e_live rounded up to 64) are written
  int32_t* status;
  unsigned long long wait_ns;   // limit of every on-chip wait
  int inject;            // opts->test_inject
  int accumulate;        // EPI_STORE_F32 (no K split, no row map): the product is added to what C holds (by reductions
                         // performed in L2: the epilogue does not read C)
  int tma_store;         // EPI_STORE_F32 (no row map, not transposed): map_c describes C (fp32, boxes of 32 x 32, 128-byte
                         // swizzle) and the epilogue stores (or adds) its blocks through shared memory with bulk tensor
                         // copies: whole 128-byte lines per row instead of 16 bytes per thread and instruction
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
// ---- CTA pairs (cluster of two; cluster_ctarank, map_to_cta, bar_arrive_cluster, cluster_sync_all: dppo_pipe.cuh) ------
// Load of one CTA of a pair; the completion bytes go to `cluster_bar`, which may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t cluster_bar) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void mma_bf16_pair(uint32_t tmem_c, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(tmem_c), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done.
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}

// Shared-memory matrix descriptor: K-major tile with rows of 128 bytes, 128-byte swizzle (8-row groups 1024 bytes apart).
__device__ __forceinline__ uint64_t make_desc_k_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);       // start address, 16-byte units
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused with swizzle): 1
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                          // layout type: 128-byte swizzle
  return d;
}
// Shared-memory matrix descriptor of an MN-major operand tile (the operand is stored [K, MN] with MN contiguous): the
// tile is a row of 64-element (128-byte) wide column blocks, each block 64 k-rows of 128 bytes (8 KB, swizzled in 8-row
// groups of 1024 bytes); consecutive blocks along MN are `block_bytes` apart.
__device__ __forceinline__ uint64_t make_desc_mn_sw128(uint32_t saddr, uint32_t block_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);       // start address, 16-byte units
  d |= (uint64_t)(block_bytes >> 4) << 16;         // leading byte offset: next 64-element block along MN
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset: next group of 8 k-rows
  d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                          // layout type: 128-byte swizzle
  return d;
}
// Instruction descriptor: D = f32, A = B = bf16, A K-major, B K-major or MN-major (bit 16), N = 256, M = 128 per CTA of
// the group (M = 256 for a pair).
__host__ __device__ constexpr uint32_t make_idesc(int cg, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn ? (1u << 16) : 0u) | ((uint32_t)(BN >> 3) << 17) |
         ((uint32_t)((BM * cg) >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16(uint32_t tmem_c, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(tmem_c), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,"
      "%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// Adds to global memory without reading it back (the addition is done by the L2 cache, the thread does not wait).
// Used where every element of the output gets exactly one contribution per launch, so nothing depends on timing.
__device__ __forceinline__ void red_add_f32x4(float* p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void red_add_f32(float* p, float a) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(a) : "memory");
}
// Bulk tensor store / reduction of one 32 x 32 fp32 block from shared memory (128-byte swizzled) into C.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// at most N of this thread's bulk groups may still be reading shared memory
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The list of work units of one CTA group.  First its whole tiles (tile = group, group + ngroups, ...).  With a
// partial-sum buffer (store epilogue) the whole tiles are those of the full waves only, and the remaining tiles (fewer
// than there are groups) are cut along K into `segs` equal segments: units (segment, tile), segment-major, dealt
// round-robin to the groups.  All units in flight at a time then belong to one or two segments and walk K in step, so
// that tiles of one row or column of the output still share their operand strips through L2; more segments fill the
// last wave better.  A segment's accumulator goes to the partial-sum slot tile * segs + segment instead of C.
constexpr int kMaxSegs = 8;
struct Plan {
  int whole;            // whole-tile units of this group
  int sk_units;         // (segment, tile) units of this group after them
  int first_sk_tile;    // tile index of the first tile of the partial wave
  int sk_tiles;         // tiles of the partial wave (0: none is cut)
  int segs, kseg;       // segments per tile, K blocks per segment
  int kblocks, group, ngroups;
  __device__ __forceinline__ int units() const { return whole + sk_units; }
  // unit i -> tile, K blocks [kb0, kb1), partial-sum slot (-1: the result goes to C)
  __device__ __forceinline__ void unit(int i, int& tile, int& kb0, int& kb1, int& slot) const {
    if (i < whole) { tile = group + i * ngroups; kb0 = 0; kb1 = kblocks; slot = -1; return; }
    const int j = group + (i - whole) * ngroups, seg = j / sk_tiles, r = j - seg * sk_tiles;
    tile = first_sk_tile + r;
    kb0 = seg * kseg;
    kb1 = kb0 + kseg < kblocks ? kb0 + kseg : kblocks;
    slot = r * segs + seg;
  }
};
template <int CG>
__device__ __forceinline__ Plan make_plan(bool allow_sk, int ntiles, int kblocks, int group, int ngroups) {
  Plan pl;
  pl.kblocks = kblocks; pl.group = group; pl.ngroups = ngroups;
  const int full_waves = ntiles / ngroups, rem = ntiles - full_waves * ngroups;
  pl.first_sk_tile = full_waves * ngroups;
  pl.sk_tiles = 0; pl.sk_units = 0; pl.segs = 1; pl.kseg = kblocks;
  // time of the partial wave with s segments, in tile times: ceil(rem * s / ngroups) / s; the smallest s within 2 % of
  // the best, and only if that saves 5 % of a tile time or more
  int best = 1;
  if (allow_sk && rem > 0) {
    float tbest = 1.f;
    for (int sgs = 2; sgs <= kMaxSegs && kblocks >= 8 * sgs; ++sgs) {
      const float t = (float)((rem * sgs + ngroups - 1) / ngroups) / (float)sgs;
      if (t < 0.98f * tbest) { tbest = t; best = sgs; }
    }
    if (tbest > 0.95f) best = 1;
  }
  if (best == 1) {
    pl.whole = group < ntiles ? (ntiles - group + ngroups - 1) / ngroups : 0;
    return pl;
  }
  pl.whole = full_waves;
  pl.sk_tiles = rem;
  pl.segs = best;
  pl.kseg = (kblocks + best - 1) / best;               // kblocks >= 8 * segs: no segment is empty
  const int total = rem * best;
  pl.sk_units = group < total ? (total - group + ngroups - 1) / ngroups : 0;
  return pl;
}

// B_MN = false: B given as [N, K] (K contiguous).  B_MN = true: B given as [K, N] (N contiguous, "NN" product); its tile is
// then loaded as boxes of 64 columns x 64 k-rows.  CG = 2: launched as clusters of two CTAs (see the top of the file).
template <int EPI, bool B_MN, int CG>
__global__ void __launch_bounds__(THREADS, 1) gemm_tn_kernel(const __grid_constant__ CUtensorMap map_a,
                                                             const __grid_constant__ CUtensorMap map_b,
                                                             const __grid_constant__ CUtensorMap map_c, Params p) {
  using C = Cfg<CG>;
  constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES, A_STAGE_BYTES = C::A_STAGE_BYTES;
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment for the 128-byte swizzle atoms (the same offset in both CTAs of a pair)
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* out_stage = smem + STAGES * STAGE_BYTES;      // 1024-byte aligned: whole swizzle atoms
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + STAGES * STAGE_BYTES + C::OUT_BYTES);
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STAGES);
  const uint32_t tfull0 = smem_u32(bars + 2 * STAGES), tempty0 = smem_u32(bars + 2 * STAGES + 2);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  const WaitCtl wc{reinterpret_cast<volatile int*>(tmem_slot + 1), p.wait_ns};
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = (CG == 2) ? cluster_ctarank() : 0u;       // 0: leader of the pair
  const int group = (CG == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int ngroups = (CG == 2) ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  if (tid == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(full0 + 8 * i, 1); mbar_init(empty0 + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tfull0 + 8 * i, 1); mbar_init(tempty0 + 8 * i, 4 * CG); }
    *wc.flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {   // the MMA warp owns the tensor memory (in a pair: the same warp of both CTAs, together)
    if (CG == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (CG == 2) cluster_sync_all();      // the peer's barriers exist before anything is sent to them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  int m_lim = p.M, k_lim = p.K;
  if (p.m_live) { const int v = *p.m_live; m_lim = v < 0 ? 0 : (v < p.M ? v : p.M); }
  if (p.k_live) { const int v = *p.k_live; k_lim = v < 0 ? 0 : (v < p.K ? v : p.K); }
  int e_lim = p.M;
  if (EPI == EPI_EXP && p.e_live) {
    const int v = *p.e_live, up = v <= 64 ? 64 : (v + 63) / 64 * 64;
    e_lim = up < p.M ? up : p.M;
  }
  const int tiles_m = m_lim > 0 ? (m_lim + C::TILE_M - 1) / C::TILE_M : (p.allow_empty ? 0 : 1), tiles_n = (p.N + BN - 1) / BN;
  const int ntiles = tiles_m * tiles_n;
  const int kblocks = k_lim > 0 ? (k_lim + BK - 1) / BK : 1;
  const Plan pl = make_plan<CG>(EPI == EPI_STORE_F32 && p.sk_part != nullptr, ntiles, kblocks, group, ngroups);
  const uint32_t smem_base = smem_u32(smem);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (of this CTA's operand slices)
    // (test injection: the producer issues nothing, so that every consumer wait of the CTA runs out)
    if (lane == 0 && !(p.inject & DPPO_INJECT_NO_COPIES)) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int u = 0; u < pl.units() && ok; ++u) {
        int tile, kb0, kb1, slot;
        pl.unit(u, tile, kb0, kb1, slot);
        const int tm = p.n_fastest ? tile / tiles_n : tile % tiles_m, tn = p.n_fastest ? tile % tiles_n : tile / tiles_m;
        const int m0 = tm * C::TILE_M + (int)rank * BM, n0 = tn * BN + (int)rank * C::B_COLS;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, wc)) { ok = false; break; }
          const uint32_t a_dst = smem_base + s * STAGE_BYTES, b_dst = a_dst + A_STAGE_BYTES;
          if (CG == 2) {
            // both CTAs' bytes are counted on the leader's barrier (the leader may post its expectation after the
            // peer's bytes have begun to land: the phase cannot complete before the leader's own arrival)
            const uint32_t bar = map_to_cta(full0 + 8 * s, 0);
            if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * s, 2 * STAGE_BYTES);
            tma_load_2d_pair(a_dst, &map_a, kb * BK, m0, bar);
            if (B_MN) {
#pragma unroll
              for (int i = 0; i < C::B_COLS / 64; ++i) tma_load_2d_pair(b_dst + i * (64 * BK * 2), &map_b, n0 + i * 64, kb * BK, bar);
            } else {
              tma_load_2d_pair(b_dst, &map_b, kb * BK, n0, bar);
            }
          } else {
            mbar_arrive_expect_tx(full0 + 8 * s, STAGE_BYTES);
            tma_load_2d(a_dst, &map_a, kb * BK, m0, full0 + 8 * s);
            if (B_MN) {
#pragma unroll
              for (int i = 0; i < C::B_COLS / 64; ++i) tma_load_2d(b_dst + i * (64 * BK * 2), &map_b, n0 + i * 64, kb * BK, full0 + 8 * s);
            } else {
              tma_load_2d(b_dst, &map_b, kb * BK, n0, full0 + 8 * s);
            }
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (in a pair: the leader's only)
    if (lane == 0 && rank == 0) {
      int s = 0;
      uint32_t ph = 0;
      uint32_t it = 0;
      bool ok = true;
      constexpr uint32_t idesc = make_idesc(CG, B_MN);
      for (int u = 0; u < pl.units() && ok; ++u, ++it) {
        int tile, kb0, kb1, slot;
        pl.unit(u, tile, kb0, kb1, slot);
        const uint32_t b = it & 1u, use = it >> 1;
        if (!mbar_wait(tempty0 + 8 * b, (use & 1u) ^ 1u, wc)) { ok = false; break; }   // epilogues drained this buffer
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_c = tmem_base + b * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full0 + 8 * s, ph, wc)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_src = smem_base + s * STAGE_BYTES, b_src = a_src + A_STAGE_BYTES;
          const uint64_t adesc = make_desc_k_sw128(a_src);
          const uint64_t bdesc = B_MN ? make_desc_mn_sw128(b_src, 64 * BK * 2) : make_desc_k_sw128(b_src);
          // per step of 16 along K: K-major operands move 32 bytes inside the swizzle atom, an MN-major one 16 k-rows (2048 bytes)
          constexpr uint64_t kStepB = B_MN ? (uint64_t)(16 * 128 >> 4) : 2ull;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if (CG == 2) mma_bf16_pair(tmem_c, adesc + (uint64_t)(k * 2), bdesc + kStepB * k, idesc, (kb != kb0 || k != 0) ? 1u : 0u);
            else mma_bf16(tmem_c, adesc + (uint64_t)(k * 2), bdesc + kStepB * k, idesc, (kb != kb0 || k != 0) ? 1u : 0u);
          }
          // stage free (in both CTAs of a pair) once these MMAs have read it
          if (CG == 2) mma_commit_pair(empty0 + 8 * s); else mma_commit(empty0 + 8 * s);
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (ok) { if (CG == 2) mma_commit_pair(tfull0 + 8 * b); else mma_commit(tfull0 + 8 * b); }   // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (TMEM lane quarter = warp % 4)
    const int q = warp & 3;
    uint32_t it = 0, out_it = 0;                 // out_it: blocks this warp has handed to bulk tensor copies
    for (int u = 0; u < pl.units(); ++u, ++it) {
      int tile, kb0, kb1, slot;
      pl.unit(u, tile, kb0, kb1, slot);
      const int tm = p.n_fastest ? tile / tiles_n : tile % tiles_m, nb = p.n_fastest ? tile % tiles_n : tile / tiles_m;
      const int m0 = tm * C::TILE_M + (int)rank * BM, n0 = nb * BN;
      const uint32_t b = it & 1u, use = it >> 1;
      const bool ok = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * b, use & 1u, wc));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int row = m0 + q * 32 + lane;
      // the gradient and exponential epilogues fill whole tiles (the rows past the live extent feed the last K block of
      // a later GEMM and must hold finite values), unless the gradient rows go through a row map
      const bool row_ok = (EPI == EPI_STORE_F32 || (EPI == EPI_GRAD && p.p_row_map)) ? row < m_lim : row < p.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + b * BN;
      if (EPI == EPI_STORE_F32 && slot >= 0) {
        // a piece of a tile's K range: the raw partial sums of this CTA's 128 rows go to the group's slot
        float* dst = p.sk_part + ((int64_t)slot * C::TILE_M + (int)rank * BM + q * 32 + lane) * BN;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
#pragma unroll
          for (int j = 0; j < 32; j += 4) *reinterpret_cast<uint4*>(dst + c + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
        }
      } else if (EPI == EPI_STORE_F32 && p.tma_store) {
        // Through shared memory: the thread writes its row's 32 columns into the warp's 32 x 32 block (16-byte pieces
        // placed by the 128-byte swizzle, so that the 32 rows of a warp do not collide on the banks), one lane hands the
        // block to a bulk tensor copy, which stores it, or adds it to C, 128 contiguous bytes per row; rows and columns
        // beyond C are clipped by the tensor map.  Two blocks per warp in turn.
        const float sc = (row_ok && p.row_scale) ? p.row_scale[row] : 1.f;
        const uint32_t wbuf = smem_u32(out_stage) + (uint32_t)q * (2u * 4096u);
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
          if (n0 + c < p.N && m0 + q * 32 < m_lim) {            // warp-uniform: the block meets C
            const uint32_t buf = wbuf + (uint32_t)(out_it & 1u) * 4096u;
            if (lane == 0 && out_it >= 2) bulk_wait_read<1>();  // the copy that read this buffer two blocks ago is done with it
            __syncwarp();
            if (p.row_scale) {
#pragma unroll
              for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * sc);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint32_t addr = buf + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) * 16);
              asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3]) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
              if (p.accumulate) tma_reduce_add_2d(&map_c, buf, n0 + c, m0 + q * 32);
              else tma_store_2d(&map_c, buf, n0 + c, m0 + q * 32);
              bulk_commit();
            }
            ++out_it;
          }
        }
      } else if (EPI == EPI_STORE_F32) {
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
          if (row_ok) {
            float* dst = p.C + (int64_t)(p.row_map ? p.row_map[row] : row) * p.ldc + n0 + c;
            if (p.row_scale) {
              const float sc = p.row_scale[row];
#pragma unroll
              for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * sc);
            }
            if (p.c_transposed) {          // the lanes of a warp hold 32 consecutive rows: 128 contiguous bytes per column
              float* ct = p.C + (int64_t)(n0 + c) * p.ldc + row;
              if (p.accumulate) {
#pragma unroll
                for (int j = 0; j < 32; ++j) if (n0 + c + j < p.N) red_add_f32(ct + (int64_t)j * p.ldc, __uint_as_float(r[j]));
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) if (n0 + c + j < p.N) ct[(int64_t)j * p.ldc] = __uint_as_float(r[j]);
              }
            } else if (p.accumulate) {
              // added to what earlier launches left (a later row block of the same dW): one contribution per element
              // and launch, launches in stream order, so the sum is the same every time
              if (n0 + c + 32 <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                  red_add_f32x4(dst + j, __uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) if (n0 + c + j < p.N) red_add_f32(dst + j, __uint_as_float(r[j]));
              }
            } else if (n0 + c + 32 <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
              for (int j = 0; j < 32; j += 4) *reinterpret_cast<uint4*>(dst + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) if (n0 + c + j < p.N) dst[j] = __uint_as_float(r[j]);
            }
          }
        }
      } else if (EPI == EPI_STATS) {
        const int a = row_ok ? p.ids[row] : -1;
        float m = -INFINITY, s = 0.f;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
          const int col0 = n0 + c;
          float vm = -INFINITY;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            float z = (col0 + j < p.N) ? __uint_as_float(r[j]) : -INFINITY;
            if (col0 + j == a) { p.z_a[row] = z; z = -INFINITY; }     // the sampled token's entry is left out of the sums
            r[j] = __float_as_uint(z);
            vm = fmaxf(vm, z);
          }
          if (vm > m) { s *= ex2((m - vm) * 1.4426950408889634f); m = vm; }
          if (m != -INFINITY) {
            const float nm = -m * 1.4426950408889634f;
            float acc = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) acc += ex2(fmaf(__uint_as_float(r[j]), 1.4426950408889634f, nm));
            s += acc;
          }
        }
        if (row_ok) p.part[(int64_t)row * tiles_n + nb] = make_float2(m, s);
      } else if (EPI == EPI_EXP) {
        const int a = row_ok ? p.ids[row] : -1;
        const float ncr = row_ok ? -p.cref2[row] : 0.f;
        const bool store = row_ok && row < e_lim;
        float s = 0.f;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
          const int col0 = n0 + c;
          if (col0 < p.N) {
            uint32_t o[16];
            float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              float v0 = ex2(fmaf(__uint_as_float(r[j]), 1.4426950408889634f, ncr));
              float v1 = ex2(fmaf(__uint_as_float(r[j + 1]), 1.4426950408889634f, ncr));
              if (col0 + j >= p.N) v0 = 0.f;
              if (col0 + j + 1 >= p.N) v1 = 0.f;
              acc0 += v0;
              acc1 += v1;
              __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
              o[j >> 1] = *reinterpret_cast<uint32_t*>(&h);
            }
            if (a >= col0 && a < col0 + 32) {      // the sampled token's entry is left out of the row's sum
              float s2 = 0.f;
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (col0 + j == a) p.z_a[row] = __uint_as_float(r[j]);
                else if (col0 + j < p.N) s2 += ex2(fmaf(__uint_as_float(r[j]), 1.4426950408889634f, ncr));
              }
              s += s2;
            } else {
              s += acc0 + acc1;
            }
            if (store) {
              __nv_bfloat16* dst = p.P + (int64_t)row * p.ldp + col0;
              if (col0 + 32 <= p.N) {
#pragma unroll
                for (int j = 0; j < 16; j += 4) *reinterpret_cast<uint4*>(dst + 2 * j) = make_uint4(o[j], o[j + 1], o[j + 2], o[j + 3]);
              } else {
                for (int j = 0; j < 32; ++j)
                  if (col0 + j < p.N) dst[j] = __ushort_as_bfloat16((unsigned short)((j & 1) ? (o[j >> 1] >> 16) : (o[j >> 1] & 0xffffu)));
              }
            }
          }
        }
        if (row_ok) p.psum[(int64_t)row * tiles_n + nb] = s;
      } else {  // EPI_GRAD
        const int a = row_ok ? p.ids[row] : -1;
        const float c2 = row_ok ? p.c2[row] : 0.f, sg = row_ok ? p.sgn[row] : 0.f, fx = row_ok ? p.fix[row] : 0.f;
        const uint32_t sign2 = (sg < 0.f) ? 0x80008000u : 0u;
        const int prow = (row_ok && p.p_row_map) ? p.p_row_map[row] : row;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c, r);
          const int col0 = n0 + c;
          if (row_ok && prow >= 0 && col0 < p.N) {
            uint32_t o[16];
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              float v0 = (sg == 0.f) ? 0.f : ex2(fmaf(__uint_as_float(r[j]), 1.4426950408889634f, c2));
              float v1 = (sg == 0.f) ? 0.f : ex2(fmaf(__uint_as_float(r[j + 1]), 1.4426950408889634f, c2));
              if (col0 + j == a) v0 = fx * sg;          // the sign flip below restores fix
              if (col0 + j + 1 == a) v1 = fx * sg;
              __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
              o[j >> 1] = (*reinterpret_cast<uint32_t*>(&h)) ^ sign2;
            }
            if (p.Pt) {
              // transposed copy: for one column the 32 lanes of the warp hold 32 consecutive rows, i.e. 64 contiguous bytes
              unsigned short* dt = reinterpret_cast<unsigned short*>(p.Pt) + (int64_t)col0 * p.ldpt + row;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) dt[(int64_t)j * p.ldpt] = (unsigned short)((j & 1) ? (o[j >> 1] >> 16) : (o[j >> 1] & 0xffffu));
            }
            __nv_bfloat16* dst = p.P + (int64_t)prow * p.ldp + col0;
            if (col0 + 32 <= p.N) {
#pragma unroll
              for (int j = 0; j < 16; j += 4) *reinterpret_cast<uint4*>(dst + 2 * j) = make_uint4(o[j], o[j + 1], o[j + 2], o[j + 3]);
            } else {
              for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) dst[j] = __ushort_as_bfloat16((unsigned short)((j & 1) ? (o[j >> 1] >> 16) : (o[j >> 1] & 0xffffu)));
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) {       // buffer drained: tell the MMA issuer (the leader's, in a pair)
        if (CG == 2 && rank != 0) bar_arrive_cluster(map_to_cta(tempty0 + 8 * b, 0));
        else mbar_arrive(tempty0 + 8 * b);
      }
    }
    // bulk tensor copies of this warp that are still under way read its shared-memory blocks: they finish first
    if (EPI == EPI_STORE_F32 && lane == 0 && out_it > 0) bulk_wait_all<0>();
  }

  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  // A CTA in which a wait ran out stays for a moment: loads it issued may still be on their way (to its own shared
  // memory and, in a pair, to the leader's barrier), and tensor-core work issued before may still be running; both
  // finish within microseconds.  A CTA that did not give up has nothing in flight: its last accumulator was read.
  if (wc.aborted()) {
    if (tid == 0 && p.status) atomicOr(p.status, DPPO_STATUS_WAIT_LIMIT);
    drain_after_abort();
  }
  // a pair leaves together: neither CTA's shared or tensor memory may go away while the other can still reach it
  if (CG == 2) cluster_sync_all();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (CG == 2) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// Second half of the K split: adds up the partial tiles that gemm_tn_kernel<EPI_STORE_F32> left in p.sk_part, group after
// segment (a fixed order: the result does not depend on timing), applies the row factor and the row map and stores the
// tile.  Launch with the same Params and the same number of CTA groups; grid = (ngroups - 1, TILE_M / 32), 256 threads.
template <int CG>
__global__ void __launch_bounds__(256) gemm_streamk_fixup_kernel(Params p, int ngroups) {
  using C = Cfg<CG>;
  int m_lim = p.M, k_lim = p.K;
  if (p.m_live) { const int v = *p.m_live; m_lim = v < 0 ? 0 : (v < p.M ? v : p.M); }
  if (p.k_live) { const int v = *p.k_live; k_lim = v < 0 ? 0 : (v < p.K ? v : p.K); }
  const int tiles_m = m_lim > 0 ? (m_lim + C::TILE_M - 1) / C::TILE_M : (p.allow_empty ? 0 : 1), tiles_n = (p.N + BN - 1) / BN;
  const int ntiles = tiles_m * tiles_n;
  const int kblocks = k_lim > 0 ? (k_lim + BK - 1) / BK : 1;
  const Plan pl = make_plan<CG>(p.sk_part != nullptr, ntiles, kblocks, 0, ngroups);
  const int r = blockIdx.x;                             // tile of the partial wave
  if (r >= pl.sk_tiles) return;
  const int tile = pl.first_sk_tile + r;
  const int tm = p.n_fastest ? tile / tiles_n : tile % tiles_m, nb = p.n_fastest ? tile % tiles_n : tile / tiles_m;
  const int lrow = blockIdx.y * 32 + (threadIdx.x >> 3);                              // row of the tile: 32 rows per block,
  const int row = tm * C::TILE_M + lrow;                                              // 8 threads per row
  if (row >= m_lim) return;
  const float sc = p.row_scale ? p.row_scale[row] : 1.f;
  float* out = p.C + (int64_t)(p.row_map ? p.row_map[row] : row) * p.ldc + nb * BN;
  for (int c4 = (threadIdx.x & 7); c4 < BN / 4; c4 += 8) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sg = 0; sg < pl.segs; ++sg) {               // segment after segment: a fixed order
      const float4 v = *reinterpret_cast<const float4*>(p.sk_part + ((int64_t)(r * pl.segs + sg) * C::TILE_M + lrow) * BN + 4 * c4);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    acc.x *= sc; acc.y *= sc; acc.z *= sc; acc.w *= sc;
    const int col = nb * BN + 4 * c4;
    if (col + 4 <= p.N && ((reinterpret_cast<uintptr_t>(out + 4 * c4) & 15) == 0)) {
      *reinterpret_cast<float4*>(out + 4 * c4) = acc;
    } else {
      const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
      for (int j = 0; j < 4; ++j) if (col + j < p.N) out[4 * c4 + j] = a4[j];
    }
  }
}

}  // namespace gemm
}  // namespace dppo
