// Small pieces shared by the row kernels that stream rows through shared-memory rings: 16-byte vectors of logits to
// floats, packed gradient stores, positions in a ring, per-row bookkeeping.
#pragma once

#include "dppo_common.cuh"

namespace dppo {

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

// Writes N gradient values starting at element j0 of an output row; `sign2` (0 or 0x80008000)
// flips the sign of every value.
template <typename OutT, int N> struct Store;
template <> struct Store<__nv_bfloat16, 8> {
  static __device__ __forceinline__ void run(__nv_bfloat16* row, uint32_t j0, const float* v, uint32_t sign2 = 0u) {
    uint4 o;
    o.x = pack_bf16x2(v[0], v[1]) ^ sign2; o.y = pack_bf16x2(v[2], v[3]) ^ sign2;
    o.z = pack_bf16x2(v[4], v[5]) ^ sign2; o.w = pack_bf16x2(v[6], v[7]) ^ sign2;
    stg128_cs(row + j0, o);
  }
};
template <> struct Store<float, 8> {
  static __device__ __forceinline__ void run(float* row, uint32_t j0, const float* v, uint32_t sign2 = 0u) {
    const uint32_t sg = sign2 & 0x80000000u;
    uint4 o0 = {__float_as_uint(v[0]) ^ sg, __float_as_uint(v[1]) ^ sg, __float_as_uint(v[2]) ^ sg, __float_as_uint(v[3]) ^ sg};
    uint4 o1 = {__float_as_uint(v[4]) ^ sg, __float_as_uint(v[5]) ^ sg, __float_as_uint(v[6]) ^ sg, __float_as_uint(v[7]) ^ sg};
    stg128_cs(row + j0, o0);
    stg128_cs(row + j0 + 4, o1);
  }
};
template <> struct Store<float, 4> {
  static __device__ __forceinline__ void run(float* row, uint32_t j0, const float* v, uint32_t sign2 = 0u) {
    const uint32_t sg = sign2 & 0x80000000u;
    uint4 o0 = {__float_as_uint(v[0]) ^ sg, __float_as_uint(v[1]) ^ sg, __float_as_uint(v[2]) ^ sg, __float_as_uint(v[3]) ^ sg};
    stg128_cs(row + j0, o0);
  }
};

struct RingPos {             // position in the endless sequence of slot uses of one ring
  int slot;
  uint32_t phase;
  __device__ __forceinline__ void advance(int nslots) {
    if (++slot == nslots) { slot = 0; phase ^= 1u; }
  }
};

// Row bookkeeping every role evaluates identically: >= 0 sampled id of a valid row, -1 row masked
// out (or past the end), -2 sampled id out of range (row treated as invalid, status bit).
__device__ __forceinline__ int load_meta(const RowParams& p, int64_t t) {
  if (t >= p.T) return -1;
  if (p.token_mask && p.token_mask[t] == 0) return -1;
  const int a = p.sampled_ids[t];
  return (a < 0 || (int64_t)a >= p.V) ? -2 : a;
}

}  // namespace dppo
