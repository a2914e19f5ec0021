// Shared device-side pieces of the DPPO loss kernels: parameter block, numeric helpers and the
// per-row scalar stage (ratio, divergence, mask, gradient coefficient).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/dppo.h"

namespace dppo {

constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.6931471805599453;

// Header of the caller's workspace, written by the prelude kernel of each call.  The accumulators are used by calls
// that finish their rows block by block (the row-block mode of the fused variant): the loss reduction of every block
// adds its rows to them, in stream order, and the last block writes the results.
struct WsHeader {
  double scale;        // s of this call
  int n_valid;         // rows with a non-zero token_mask byte
  int pad0;
  double acc[6];       // loss, sum D, sum |pi(a) - mu(a)|, sum r, sum |loss term|, blocked rows
  float max_d;
  int pad1[15];
};
static_assert(sizeof(WsHeader) == 128, "WsHeader layout");

struct RowParams {
  const void* logits;
  int64_t T, V, ld_in;
  const int32_t* sampled_ids;
  const float* mu_logp;
  const int32_t* topk_ids;
  const float* topk_p;
  const float* adv;
  const uint8_t* token_mask;
  int variant, K;
  float delta;
  float loss_scale;          // > 0: caller's s
  float is_cap;              // C of Eq. unified_grad (<= 0 or inf: none)
  float eps_low;             // lower clip range of DPPO_PPO_CLIP (<= 0: delta)
  unsigned long long wait_ns;  // limit of every on-chip wait
  int inject;                // opts->test_inject
  int row_cluster;           // opts->row_cluster (ring kernel: 0 = automatic)
  void* dlogits;
  int64_t ld_out;
  float* divergence;
  uint8_t* mask;
  float* loss;
  float* stats;
  int32_t* status;
  WsHeader* hdr;             // workspace
  float* row_loss;           // [T] -s M r A
  float* row_r;              // [T] r_t
  float* row_absdiff;        // [T] |pi(a) - mu(a)|
};

// What the scalar stage hands to the gradient sweep of one row.
struct RowCoef {
  float c2;       // exponent offset: dlogits_j = sgn * 2^(z_j*log2e + c2) for j != a
  float sgn;      // +1 / -1 (sign of g); 0 when the whole row is zero
  float fix;      // value of dlogits at j = a
  int zero_row;   // 1: write zeros (invalid row, blocked row, zero advantage)
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Merge two online-softmax partials (m, s): s counts exp(z - m).  -inf maxima carry s = 0.
__device__ __forceinline__ void merge_ms(float& m, float& s, float m2, float s2) {
  float mn = fmaxf(m, m2);
  float ref = (mn == -INFINITY) ? 0.f : mn;
  s = s * ex2_approx((m - ref) * kLog2e) + s2 * ex2_approx((m2 - ref) * kLog2e);
  m = mn;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ double xlogx_over_y(double x, double y) {
  if (x <= 0.0) return 0.0;
  if (y <= 0.0) return INFINITY;
  return x * (log(x) - log(y));
}

// Log-sum-exp of a row from the sum over all entries but the sampled one, kept apart so that 1 - pi(a) stays
// accurate to the relative precision of that sum when pi(a) is close to 1 (1 - exp(z_a - lse) would cancel):
//   m_o, S_o   maximum and sum of exp(z_j - m_o) over j != a (m_o = -inf, S_o = 0 if there is no such mass)
//   z_a        the sampled token's logit
// Gives lse over the whole row and log_other = log sum_{j != a} exp(z_j), so that log(1 - pi(a)) = log_other - lse.
__device__ __forceinline__ void combine_lse(double m_o, double S_o, double z_a, double& lse, double& log_other) {
  const bool have_o = (S_o > 0.0) || (S_o != S_o);         // a NaN sum (a NaN logit) is carried into lse
  log_other = have_o ? m_o + log(S_o) : -INFINITY;
  if (z_a != z_a) { lse = NAN; return; }
  const double M = fmax(have_o ? m_o : -INFINITY, z_a);
  if (M == -INFINITY || M == INFINITY) { lse = M; return; }   // no mass at all / an infinite logit: not finite, the caller reports it
  lse = M + log((have_o ? S_o * exp(m_o - M) : 0.0) + exp(z_a - M));
}

// Per-row scalar stage, run by ONE full warp (all 32 lanes call it with the same arguments).
//   lse        log-sum-exp of the row (double, from fp32 partial sums)
//   log_other  log of the sum of exp(z_j) over j != a (see combine_lse)
//   z_at(id, k)  fp32 value of this row's logit `id`; k is its position in the top-K list, -1 for the sampled id
//   list_at(k, id, pm)  entry k of the row's top-K list (id and rollout probability); a caller that fetched the list
//                earlier hands it over here, the default reads it from global memory
// Returns on every lane the same values.  `flags` receives DPPO_STATUS_* bits found here.
template <typename ZAt, typename ListAt>
__device__ __forceinline__ void row_scalars_warp(const RowParams& p, int64_t t, int a, double lse, double log_other, double scale,
                                                 ZAt z_at, ListAt list_at, float& D_out, int& M_out, double& g_out,
                                                 float& r_out, float& absdiff_out, double& pi_a_out, int& flags) {
  const int lane = threadIdx.x & 31;
  const double mu_logp = (double)p.mu_logp[t];
  const double adv = (double)p.adv[t];
  const double lpa = (double)z_at(a, -1) - lse;           // log pi(a_t)
  const double pi_a = exp(lpa);
  const double mu_a = exp(mu_logp);
  const double r = exp(lpa - mu_logp);                // Eq. ppo-clip
  double D;
  bool ppo_blocked = false;
  if (p.variant == DPPO_PPO_CLIP) {                   // baseline: ratio clipping (App. C.1), D reported as |r - 1|
    D = fabs(r - 1.0);
    const double eh = (double)p.delta, el = (p.eps_low > 0.f) ? (double)p.eps_low : (double)p.delta;
    ppo_blocked = (adv > 0.0 && r - 1.0 > eh) || (adv < 0.0 && 1.0 - r > el);
  } else if (p.variant == DPPO_MINIMAL_MASK) {        // ablation of Sec. 5.3: signed drop of the sampled token's probability
    D = mu_a - pi_a;
    ppo_blocked = (adv < 0.0 && D >= (double)p.delta);
  } else if (p.variant == DPPO_GIVEN_D) {             // the caller's divergence of this token (read before it is written back)
    D = (double)p.divergence[t];
  } else if (p.variant == DPPO_BINARY_TV) {
    D = fabs(mu_a - pi_a);                            // Eq. binary_tv
  } else if (p.variant == DPPO_BINARY_KL) {           // Eq. binary_kl
    double first = (mu_a > 0.0) ? mu_a * (mu_logp - lpa) : 0.0;
    // (1 - mu(a)) log((1 - mu(a)) / (1 - pi(a))) with log(1 - pi(a)) = log_other - lse
    const double om_a = -expm1(mu_logp);
    double second = 0.0;
    if (om_a > 0.0) second = (log_other == -INFINITY) ? INFINITY : om_a * (log(om_a) - (log_other - lse));
    D = first + second;
  } else {
    // Reduced categorical over set(top-K ids) u {a} u {other}  (Sec. 4.4, Eq. topk_tv / topk_kl)
    // per list entry in fp32 (log pi from the double lse, then expf / logf: relative error ~1e-7, two orders below the
    // tolerance of D); the lane's partial sums go to double for the reduction across the warp
    // (the two mass sums in double: a lane may hold a probability close to 1 next to a tiny one)
    double l_mu = 0.0, l_pi = 0.0;
    float l_tv = 0.f, l_kl = 0.f;
    int in_list = 0, bad = 0;
    for (int k = lane; k < p.K; k += 32) {
      int id;
      float pm;
      list_at(k, id, pm);
      if (id < 0 || (int64_t)id >= p.V) { bad = 1; continue; }
      const float lpk = (float)((double)z_at(id, k) - lse);
      const float pk = expf(lpk);
      l_mu += (double)pm;
      if (id != a) l_pi += (double)pk;                     // pi's mass on the list without the sampled token
      l_tv += fabsf(pm - pk);
      if (pm > 0.f) l_kl += pm * (logf(pm) - lpk);
      in_list |= (id == a);
    }
    double sum_mu = warp_sum(l_mu), sum_pi = warp_sum(l_pi), tv = warp_sum((double)l_tv), kl = warp_sum((double)l_kl);
    in_list = __any_sync(0xffffffffu, in_list);
    bad = __any_sync(0xffffffffu, bad);
    if (bad) flags |= DPPO_STATUS_BAD_TOPK_ID;
    if (!in_list) {
      sum_mu += mu_a;
      tv += fabs(mu_a - pi_a);
      if (mu_a > 0.0) kl += mu_a * (mu_logp - lpa);
    }
    double om = 0.0, op = 0.0, op_raw = 0.0;           // "other" bucket; empty when the set is the vocabulary
    if ((int64_t)p.K + (in_list ? 0 : 1) < p.V) {
      om = fmin(1.0, fmax(0.0, 1.0 - sum_mu));
      // 1 - sum of pi over the set = (1 - pi(a)) - pi's mass on the rest of the list, with 1 - pi(a) taken from the
      // sum over the other entries (no cancellation when pi(a) is close to 1)
      op_raw = exp(log_other - lse) - sum_pi;
      op = fmin(1.0, fmax(0.0, op_raw));
    }
    if (p.variant == DPPO_TOPK_TV) {
      D = 0.5 * (tv + fabs(om - op));
    } else {
      // When a token of the list other than the sampled one holds nearly all of pi's mass, the difference above is
      // below what a normaliser summed in fp32 resolves (about 1e-7 absolute) and may come out as zero or negative while
      // the rollout's own remainder is just as small: that is rounding, not a token that pi excludes, and the bucket's
      // term, at most of the order of that remainder, is then left out instead of being reported as +inf.
      const bool unresolved = (op_raw <= 0.0) && (op_raw > -1e-5) && (om < 1e-5);
      D = kl + (unresolved ? 0.0 : xlogx_over_y(om, op));
    }
  }
  // Eq. dppo_obj: blocked iff D > delta and the ratio already left 1 on the side the advantage pushes.
  const bool away = (adv > 0.0 && lpa > mu_logp) || (adv < 0.0 && lpa < mu_logp);
  const int M = (p.variant == DPPO_PPO_CLIP || p.variant == DPPO_MINIMAL_MASK) ? (ppo_blocked ? 0 : 1) : ((away && D > (double)p.delta) ? 0 : 1);
  // Eq. unified_grad: the importance weight in loss and gradient is min(r, C)
  const double w = (p.is_cap > 0.f && isfinite(p.is_cap)) ? fmin(r, (double)p.is_cap) : r;
  D_out = (float)D;
  M_out = M;
  g_out = scale * (double)M * w * adv;
  r_out = (float)r;
  absdiff_out = (float)fabs(mu_a - pi_a);
  pi_a_out = pi_a;
}

template <typename ZAt>
__device__ __forceinline__ void row_scalars_warp(const RowParams& p, int64_t t, int a, double lse, double log_other, double scale,
                                                 ZAt z_at, float& D_out, int& M_out, double& g_out,
                                                 float& r_out, float& absdiff_out, double& pi_a_out, int& flags) {
  const int32_t* ids = p.topk_ids + t * (int64_t)p.K;
  const float* ps = p.topk_p + t * (int64_t)p.K;
  auto list_at = [&](int k, int& id, float& pm) { id = ids[k]; pm = ps[k]; };
  row_scalars_warp(p, t, a, lse, log_other, scale, z_at, list_at, D_out, M_out, g_out, r_out, absdiff_out, pi_a_out, flags);
}

// Turns g, lse into the coefficients of the gradient sweep.
__device__ __forceinline__ RowCoef make_coef(double g, double lse, double pi_a) {
  RowCoef c;
  if (g == 0.0) {
    c.c2 = 0.f; c.sgn = 0.f; c.fix = 0.f; c.zero_row = 1;
    return c;
  }
  c.zero_row = 0;
  c.sgn = (g > 0.0) ? 1.f : -1.f;
  c.c2 = (float)((log(fabs(g)) - lse) / kLn2);
  c.fix = (float)(g * (pi_a - 1.0));
  return c;
}

// Launchers implemented in the kernel files.
cudaError_t launch_prelude(const RowParams& p, cudaStream_t st);
// block_first / block_last: position of these rows in a call that finishes its rows block by block (both true: the
// whole call at once); the totals of earlier blocks wait in the workspace header
cudaError_t launch_finalize(const RowParams& p, cudaStream_t st, bool block_first = true, bool block_last = true);
cudaError_t launch_generic(const RowParams& p, int in_dtype, int out_dtype, cudaStream_t st);
cudaError_t launch_ring(const RowParams& p, int in_dtype, int out_dtype, cudaStream_t st);
bool ring_layout_ok(const RowParams& p, int in_dtype, int out_dtype);

}  // namespace dppo
