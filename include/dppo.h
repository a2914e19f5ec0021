/*
 * dppo.h - C ABI of the DPPO per-token loss path for NVIDIA B200 (sm_100a).
 *
 * DPPO (Divergence Proximal Policy Optimization, "Rethinking the Trust Region
 * in LLM Reinforcement Learning") replaces PPO's ratio clipping by a mask that
 * depends on an estimate D_t of the divergence between the rollout policy mu
 * and the trainer policy pi at every response token.  For each token row this
 * library streams the trainer's vocabulary logits once and produces
 *
 *   lse_t      = log sum_j exp(z_tj)                      (Sec. 3: pi is a categorical over the vocabulary)
 *   r_t        = pi(a_t) / mu(a_t)                        (Eq. ppo-clip)
 *   D_t        = Binary-TV / Binary-KL / TopK-TV / TopK-KL (Eq. binary_tv, binary_kl, topk_tv, topk_kl)
 *   M_t        = 0 iff D_t > delta and the update moves r_t away from 1
 *                in the direction the advantage pushes     (Eq. dppo_obj)
 *   loss       = -s * sum_t M_t r_t A_t                   (Eq. dppo_obj, as a loss to minimise)
 *   dlogits_tj = s M_t r_t A_t (pi_tj - 1[j = a_t])       (Eq. unified_grad with C = infinity)
 *
 * without ever materialising a probability tensor.
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Unless a parameter says "host", every pointer is a DEVICE pointer owned by
 *    the caller.  The library allocates nothing and keeps no state between calls
 *    (every switch is a field of dppo_opts, per call; the one exception is the
 *    built-in scratch array of dppo_loss_fwd_bwd_static_ws, see there).  It
 *    enqueues its kernels on `cuda_stream` (a cudaStream_t passed as void*,
 *    NULL = the default stream) and never synchronises.
 *  - Range checks of the ids and the test for a finite log-sum-exp are always on
 *    (they cost nothing next to the row's traffic); there is no switch for them.
 *  - Return value: DPPO_OK (0) when the kernels were enqueued; a negative
 *    DPPO_ERR_* code for misuse the host can see, in which case nothing was
 *    launched.  dppo_error_string() names a code.
 *  - Anomalies only the device can see never trap: they OR bits into *status
 *    (DPPO_STATUS_*), and the offending row is treated as invalid (D = 0, M = 0,
 *    zero gradient row, no loss term).  The caller zeroes *status beforehand.
 *  - Results are deterministic: the same inputs give bit-identical outputs.
 *  - Rows whose token_mask byte is 0 are never read; their outputs are zero.
 *  - The scale s is opts->loss_scale when that is > 0, otherwise 1 / N_valid
 *    with N_valid the number of rows of THIS call whose token_mask is non-zero
 *    (0 if there is none, so an empty or fully masked call returns loss = 0).
 */
#ifndef DPPO_H_
#define DPPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Divergence approximations (Sec. 4.4: Binary and Top-K approximation). */
enum { DPPO_BINARY_TV = 0, DPPO_BINARY_KL = 1, DPPO_TOPK_TV = 2, DPPO_TOPK_KL = 3,
       /* baseline the paper compares against: D_t = |r_t - 1| with the PPO / GRPO ratio-clip mask (App. C.1):
          M_t = 0 iff (A > 0 and r - 1 > delta) or (A < 0 and 1 - r > eps_low); delta plays eps_high */
       DPPO_PPO_CLIP = 4,
       /* ablation of Sec. 5.3: D_t = mu(a_t) - pi(a_t) (signed), M_t = 0 iff A_t < 0 and D_t >= delta */
       DPPO_MINIMAL_MASK = 5,
       /* Eq. dppo_obj with a per-token divergence computed elsewhere, e.g. the exact full-vocabulary TV or KL that the
          forms of Sec. 4.4 approximate (dppo_exact_divergence): the caller fills `divergence` with D_t before the call;
          mask, loss and gradient follow as for the other variants.  Device entry points only. */
       DPPO_GIVEN_D = 6 };
/* Element types of the logits / dlogits tensors. */
enum { DPPO_F32 = 0, DPPO_BF16 = 1 };
/* opts->dlogits_dtype */
enum { DPPO_DLOGITS_SAME = 0, DPPO_DLOGITS_F32 = 1 };
/* opts->kernel.  RING: the bulk-copy (TMA) streaming kernel; it takes logits / dlogits whose bases are 16-byte aligned
 * and whose rows either all start on 16-byte boundaries with V * element size a multiple of 16, or are shifted alike
 * (same element size, row strides in bytes equal modulo 16: e.g. both contiguous with an odd V).  GENERIC: element-wise
 * kernel for any layout (several times slower).  AUTO picks RING whenever it can take the layout. */
enum { DPPO_KERNEL_AUTO = 0, DPPO_KERNEL_GENERIC = 1, DPPO_KERNEL_RING = 2 };
/* opts->test_inject (testing only).  NO_COPIES: the copy producers of the kernels issue nothing, so that every on-chip
 * wait for data runs out after opts->wait_limit_us and the call returns with DPPO_STATUS_WAIT_LIMIT set and undefined
 * results; nothing faults or hangs, and the next call works normally.  It exists so that the give-up path of the
 * bounded waits can be exercised. */
enum { DPPO_INJECT_NO_COPIES = 1 };

/* Host-visible error codes. */
enum {
  DPPO_OK = 0,
  DPPO_ERR_NULL = -1,        /* a required pointer is NULL                                  */
  DPPO_ERR_SHAPE = -2,       /* T < 0, V < 1, K < 0, K > V, d < 1                            */
  DPPO_ERR_DTYPE = -3,       /* unknown logits / dlogits dtype                               */
  DPPO_ERR_VARIANT = -4,     /* unknown variant                                              */
  DPPO_ERR_TOPK = -5,        /* Top-K variant with K > 0 but a NULL id / probability list    */
  DPPO_ERR_STRIDE = -6,      /* a row stride smaller than V                                  */
  DPPO_ERR_ALIGN = -7,       /* pointer / stride alignment the requested kernel cannot take  */
  DPPO_ERR_WORKSPACE = -8,   /* workspace NULL, misaligned or smaller than dppo_workspace_bytes */
  DPPO_ERR_ALIAS = -9,       /* dlogits overlaps logits without being the same tensor in place (same base, element size, stride) */
  DPPO_ERR_CUDA = -10,       /* a CUDA runtime call failed (launch, copy)                    */
  DPPO_ERR_UNSUPPORTED = -11, /* combination not implemented                                 */
  DPPO_ERR_TOO_MANY_ROWS = -12 /* T above DPPO_STATIC_WS_MAX_ROWS (dppo_loss_fwd_bwd_static_ws)  */
};

/* Bits OR-ed into *status by the device. */
enum {
  DPPO_STATUS_BAD_SAMPLED_ID = 1, /* sampled_ids[t] outside [0, V)          */
  DPPO_STATUS_BAD_TOPK_ID = 2,    /* a mu_topk_ids entry outside [0, V)     */
  DPPO_STATUS_NONFINITE_ROW = 4,  /* lse of a row is NaN or infinite         */
  DPPO_STATUS_WAIT_LIMIT = 8      /* a bounded on-chip wait gave up          */
};

/* Options; all-zero means defaults. */
typedef struct dppo_opts {
  float loss_scale;    /* s > 0: use it (e.g. a global 1/N for micro-batched or sharded calls);
                          <= 0: s = 1 / N_valid of this call (token mean)                       */
  int dlogits_dtype;   /* DPPO_DLOGITS_SAME: dlogits has the logits dtype; DPPO_DLOGITS_F32      */
  int kernel;          /* DPPO_KERNEL_AUTO picks the shared-memory ring kernel when the layout
                          allows 16-byte bulk copies and the scalar kernel otherwise            */
  float is_cap;        /* C of Eq. unified_grad: the importance weight in loss and gradient is min(r_t, C);
                          <= 0 or +inf: no truncation (Eq. dppo_obj).  The paper's scaling runs use C = 5,
                          CISPO / PG-TIS is C = 3 with delta = +inf (no mask)                            */
  float eps_low;       /* DPPO_PPO_CLIP only: lower clip range; <= 0: same as delta                      */
  int lm_head_layout;  /* dppo_fused_lmhead_fwd_bwd only: DPPO_LM_HEAD_DV (0) = W and dW are [d, V] row-major;
                          DPPO_LM_HEAD_VD (1) = both are [V, d] row-major (how a linear layer stores its weight)  */
  int gemm_cta_group;  /* tensor-core GEMMs (fused variant, dppo_gemm_*): 0 or 2 = 256 x 256 tiles on pairs of SMs
                          (tcgen05 cta_group::2, each SM stages half of the B tile); 1 = 128 x 256 tiles on single SMs.
                          The results of the two modes agree up to the order of the fp32 additions in the tensor cores */
  int fused_rows_per_block;  /* dppo_fused_lmhead_fwd_bwd only: R > 0 finishes the rows in blocks of R (forward, scalars,
                          dHidden, dW += per block, with the scale s and N_valid of the whole call), so that the
                          workspace is that of min(T, R) rows whatever T is; 0 = all rows at once.  Multiples of 256
                          use the tensor-core tiles best */
  int wait_limit_us;   /* how long one on-chip wait (for a copy, for another warp) may take before the kernel gives up
                          and sets DPPO_STATUS_WAIT_LIMIT, in microseconds; 0 = about 2 s.  Waits normally take
                          microseconds; the limit only bounds the damage of a lost copy */
  int test_inject;     /* DPPO_INJECT_* bits, testing only; 0 in production                                          */
  int fused_two_pass;  /* dppo_fused_lmhead_fwd_bwd only: 1 = every row takes the two-pass route (statistics GEMM, then a
                          second GEMM over the same tiles that writes the finished bf16 gradient), which rounds dlogits once,
                          so that dW carries one bf16 rounding instead of two (|error| <= 2^-8 |hidden|^T |dlogits|), at the
                          price of computing every logits tile twice (about a third more time); 0 = single pass          */
  int row_cluster;     /* ring kernel of dppo_loss_fwd_bwd: SMs that share a row (each streams every n-th 16 KB chunk of it
                          and the per-row sums are exchanged through distributed shared memory).  0 = automatic: 1 for rows
                          of up to 20 chunks (V <= 163 840 bf16), 2 up to 64 chunks, then 4, so that the rows in flight
                          between their first and second read still fit L2; 1, 2, 4 = forced.  Results do not depend on it
                          beyond the order of the fp32 additions in the row sums */
} dppo_opts;
enum { DPPO_LM_HEAD_DV = 0, DPPO_LM_HEAD_VD = 1 };

/* Bytes of device scratch dppo_loss_fwd_bwd needs for a call of this shape (256-byte aligned pointer expected;
 * today a function of T alone: a header and three fp32 values per row).  Contents need no initialisation and carry
 * nothing between calls. */
size_t dppo_workspace_bytes(int64_t T, int64_t V, int K, int variant);

/*
 * Forward + backward of the DPPO loss over T token rows (Eq. dppo_obj; gradient:
 * Eq. unified_grad with C = infinity, the mask not differentiated).
 *
 *  logits          [T, V] row-major with row stride `logits_row_stride` elements (>= V),
 *                  dtype `logits_dtype` (DPPO_F32 or DPPO_BF16).
 *  sampled_ids     [T] token a_t sampled by the rollout policy.
 *  mu_logp         [T] log mu(a_t | s_t) stored by the rollout engine; always required (r_t needs it).
 *  mu_topk_ids     [T, K] ids of the rollout policy's K most probable tokens (any order, no
 *                  duplicates), and
 *  mu_topk_p       [T, K] their probabilities under mu; both may be NULL when K == 0 or for the
 *                  Binary variants.  The reduced distribution is over set(mu_topk_ids) u {a_t}
 *                  plus one "other" bucket (Sec. 4.4); a_t uses the list's probability when it is
 *                  a member and exp(mu_logp) otherwise.
 *  advantages      [T] per-token advantage A_t.
 *  token_mask      [T] bytes, non-zero = valid row; NULL = all rows valid.
 *  variant, K, delta   divergence approximation, list width, threshold (mask test is D_t > delta).  delta = +inf
 *                  disables the mask (the PG-IS / CISPO baselines of App. C.1).
 *  opts            NULL = defaults.
 *  loss            [1]  out: -s * sum_t M_t r_t A_t.
 *  divergence      [T]  out: D_t (0 for invalid rows; +inf possible for KL when pi puts zero mass
 *                  where mu does not).  With DPPO_GIVEN_D it is also an input: D_t of every row on entry; on
 *                  return the values of valid rows are unchanged, rows that were dropped read 0.
 *  mask            [T]  out: M_t as bytes (0 for invalid rows).
 *  dlogits         [T, V] out, row stride `dlogits_row_stride` (>= V), dtype per opts; may be the
 *                  same buffer as logits (in place) when the element sizes match and the strides
 *                  are equal; any other overlap of the two tensors is rejected (DPPO_ERR_ALIAS).
 *  stats           [8] out or NULL: N_valid, N_blocked (valid rows with M = 0), sum D, max D,
 *                  sum |pi(a)-mu(a)|, sum r, sum |loss term|, reserved.  Sums skip non-finite D.
 *  status          [1] in/out device word, see DPPO_STATUS_*.
 *  workspace       device scratch of at least dppo_workspace_bytes(T, V, K, variant) bytes.
 */
int dppo_loss_fwd_bwd(const void* logits, int64_t T, int64_t V, int64_t logits_row_stride, int logits_dtype,
                      const int32_t* sampled_ids, const float* mu_logp,
                      const int32_t* mu_topk_ids, const float* mu_topk_p,
                      const float* advantages, const uint8_t* token_mask,
                      int variant, int K, float delta, const dppo_opts* opts,
                      float* loss, float* divergence, uint8_t* mask,
                      void* dlogits, int64_t dlogits_row_stride,
                      float* stats, int32_t* status,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Bytes of device staging dppo_loss_fwd_bwd_host needs (inputs, outputs and workspace for
 * `rows_per_chunk` rows at a time, two chunks in flight). */
size_t dppo_host_staging_bytes(int64_t rows_per_chunk, int64_t V, int K, int logits_dtype, int dlogits_dtype);

/*
 * The same operation on HOST buffers (pinned memory recommended): rows are copied to the device
 * in chunks of `rows_per_chunk`, processed, and the per-token outputs copied back, with the
 * copies of one chunk overlapping the kernels of the other on two internal streams.  Pointer
 * arguments with the same names as above have the same meaning but are HOST pointers
 * (contiguous rows: stride V).  `dlogits_host` [T, V] receives the gradient (its copy back to the
 * host overlaps the next chunk's copy to the device); it may be NULL when only loss, divergence and
 * mask are wanted, in which case the gradient is computed and dropped.  `staging` is DEVICE memory
 * of at least dppo_host_staging_bytes(...) bytes, 256-byte aligned, owned by the caller.
 * `status_host` receives the OR of the device status words.  Because the token-mean scale needs
 * N_valid of the whole batch before the first chunk, it is counted on the host from token_mask.
 * The call synchronises with the device before returning (the results are on the host).
 * Creates and destroys two CUDA streams and an event per call; allocates no device memory.
 * Any number of chunks is fine (the chunks' losses are collected every few thousand chunks).
 */
int dppo_loss_fwd_bwd_host(const void* logits, int64_t T, int64_t V, int logits_dtype,
                           const int32_t* sampled_ids, const float* mu_logp,
                           const int32_t* mu_topk_ids, const float* mu_topk_p,
                           const float* advantages, const uint8_t* token_mask,
                           int variant, int K, float delta, const dppo_opts* opts,
                           float* loss_host, float* divergence_host, uint8_t* mask_host,
                           void* dlogits_host, int32_t* status_host,
                           void* staging, size_t staging_bytes, int64_t rows_per_chunk);

/*
 * dppo_loss_fwd_bwd for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this entry point; it exists for integration only.)
 *
 * Who needs it: code that runs where every byte of device memory already belongs to someone else,
 * for instance a trainer whose framework allocator claimed the whole GPU at start-up, so that a
 * cudaMalloc for the scratch may fail, or a step loop that must not call cudaMalloc / cudaFree
 * because those calls stall the whole device.  Such a caller still owns its inputs and outputs, but
 * has nowhere to get the `workspace` of dppo_loss_fwd_bwd from.
 *
 * Here the scratch is a fixed array inside the library image (256 + 12 * DPPO_STATIC_WS_MAX_ROWS
 * bytes, about 0.75 MiB), present on every GPU that loads the library until the process exits.
 * The call allocates nothing and frees nothing.  All other arguments, results, status bits and
 * error codes are those of dppo_loss_fwd_bwd, with these differences:
 *   - T may not exceed DPPO_STATIC_WS_MAX_ROWS; a larger T returns DPPO_ERR_TOO_MANY_ROWS and
 *     launches nothing (split the batch and pass opts->loss_scale, as for micro-batches).
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and keeps it for the life of the process.  Make that first call outside any
 *     stream capture, and do not use this entry point again after a cudaDeviceReset.
 *   - All calls on one device share the one array.  Nothing in it needs clearing: each call
 *     rewrites what it reads, and what the previous call left behind is ignored.  Two calls
 *     whose kernels can overlap on the GPU (different streams, no dependency) race on it and give
 *     undefined results; keep such calls on one stream or order them with events.
 */
#define DPPO_STATIC_WS_MAX_ROWS 65536
int dppo_loss_fwd_bwd_static_ws(const void* logits, int64_t T, int64_t V, int64_t logits_row_stride, int logits_dtype,
                                const int32_t* sampled_ids, const float* mu_logp,
                                const int32_t* mu_topk_ids, const float* mu_topk_p,
                                const float* advantages, const uint8_t* token_mask,
                                int variant, int K, float delta, const dppo_opts* opts,
                                float* loss, float* divergence, uint8_t* mask,
                                void* dlogits, int64_t dlogits_row_stride,
                                float* stats, int32_t* status, void* cuda_stream);

/* Bytes of device workspace dppo_fused_lmhead_fwd_bwd needs (256-byte aligned pointer expected). */
size_t dppo_fused_workspace_bytes(int64_t T, int64_t d, int64_t V, int K);

/*
 * Fused LM-head variant (not in the paper, which takes the trainer's logits as given; the loss is Eq. dppo_obj
 * with any of the divergence approximations of Sec. 4.4, the gradient Eq. unified_grad):
 * logits = hidden x W are produced tile by tile on the tensor cores and consumed in the accumulator epilogue, so the
 * [T, V] logits are never written to memory; the gradient is propagated to hidden and W.
 *
 *  hidden   [T, d] bf16 row-major;  W  [d, V] bf16 row-major (LM head);  d and V multiples of 8, 16-byte aligned.
 *           With opts->lm_head_layout = DPPO_LM_HEAD_VD, W is [V, d] row-major and dW is written as [V, d] too
 *           (no transposed copy is made: the operands are read, and dW is stored, in that layout directly).
 *  sampled_ids, mu_logp, advantages, token_mask, delta, opts, loss, divergence, mask, stats, status: as for
 *           dppo_loss_fwd_bwd.  mu_topk_ids / mu_topk_p [T, K]: as for dppo_loss_fwd_bwd (Top-K variants; the K
 *           logits per row are computed as dot products, K is ignored by the other variants).
 *  dHidden  [T, d] fp32 out: d loss / d hidden = dlogits . W^T.
 *  dW       [d, V] fp32 out: d loss / d W = hidden^T . dlogits (overwritten, not accumulated).
 *  workspace  device scratch of at least dppo_fused_workspace_bytes(T, d, V, K) bytes; it holds packed copies of hidden
 *           and the bf16 exponentials of the logits (about 2 T V bytes; plus W^T, 2 d V bytes, for Top-K variants).
 *           With opts->fused_rows_per_block = R > 0 the rows are finished R at a time and the workspace needed is
 *           dppo_fused_workspace_bytes(min(T, R), d, V, K), whatever T is: nothing of size T x V is ever staged.  The
 *           results are the same up to the order in which the blocks' contributions to dW are added (fixed: block
 *           after block), and repeated calls give identical bits.
 * Every logits tile is computed once: the forward GEMM writes exp(z - c_t) in bf16 against a per-row reference known
 * beforehand (c_t = the sampled token's logit) together with the fp32 row sums; the per-row factor g_t / S_t that turns
 * those exponentials into the gradient with respect to the logits is applied to the rows of dHidden in fp32 and to the
 * hidden rows (bf16) in front of the dW GEMM.  Entrywise accuracy: |error of dHidden| <= 2^-8 |dlogits| |W|^T,
 * |error of dW| <= 2^-7 |hidden|^T |dlogits| (one resp. two bf16 roundings, fp32 accumulation).  Rows for which the
 * reference is unusable (pi(a_t) below 2^-60, non-finite logits) are recomputed by a two-pass route inside the same
 * call; non-finite rows raise DPPO_STATUS_NONFINITE_ROW and are dropped.
 * Rows with token_mask 0 are left out of every GEMM, rows with zero advantage out of the two backward GEMMs: the
 * remaining rows are packed on the device, their count is never read by the host, and the call stays asynchronous.
 * The outputs are the same as without packing: such rows of dHidden are zero.
 */
int dppo_fused_lmhead_fwd_bwd(const void* hidden, const void* W, int64_t T, int64_t d, int64_t V,
                              const int32_t* sampled_ids, const float* mu_logp,
                              const int32_t* mu_topk_ids, const float* mu_topk_p, const float* advantages,
                              const uint8_t* token_mask, int variant, int K, float delta, const dppo_opts* opts,
                              float* loss, float* divergence, uint8_t* mask, float* dHidden, float* dW,
                              float* stats, int32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The tensor-core GEMM the fused variant is built from, exposed for testing and reuse:
 * C[M, N] (fp32, row stride ldc) = A[M, K] . B[N, K]^T with A and B bf16 row-major (row strides lda, ldb elements,
 * multiples of 8; 16-byte aligned bases), fp32 accumulation.  status: device word, DPPO_STATUS_WAIT_LIMIT on a
 * bounded wait that ran out (may be NULL).  opts (NULL = defaults): gemm_cta_group, wait_limit_us, test_inject.
 */
int dppo_gemm_tn_bf16(const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K, float* C, int64_t ldc,
                      int32_t* status, const dppo_opts* opts, void* cuda_stream);

/* The same with B given as [K, N] row-major (N contiguous, row stride ldb): C[M, N] = A[M, K] . B[K, N]. */
int dppo_gemm_nn_bf16(const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K, float* C, int64_t ldc,
                      int32_t* status, const dppo_opts* opts, void* cuda_stream);

/*
 * Exact full-vocabulary divergence between the rollout policy and the trainer policy, and the trainer policy's
 * entropy, streamed from the two logits tensors (App. B defines the exact TV and KL that the Binary / Top-K forms bound
 * from below; App. E lists entropy and |pi - mu| among the run metrics).  No probability tensor is materialised.
 *
 *  logits, mu_logits  [T, V] row-major (row strides in elements, >= V), both of `dtype` (DPPO_F32 or DPPO_BF16).
 *  token_mask         [T] bytes or NULL; rows with a zero byte are not read and give 0.
 *  tv, kl, entropy    [T] out: 1/2 sum_j |mu_j - pi_j|,  sum_j mu_j log(mu_j / pi_j),  -sum_j pi_j log pi_j.
 *                     tv may be NULL: KL and entropy are complete after one sweep over the two rows, only the TV needs a
 *                     second one (with both normalisers known), which is then left out.
 *  status             device word; DPPO_STATUS_NONFINITE_ROW if a row's log-sum-exp is not finite (outputs 0).
 *  opts               NULL = defaults; wait_limit_us and test_inject are the fields that apply.
 * Needs no workspace.  With a TV output each row is read twice (the second time normally from L2), without it once.
 */
int dppo_exact_divergence(const void* logits, const void* mu_logits, int64_t T, int64_t V,
                          int64_t logits_row_stride, int64_t mu_row_stride, int dtype,
                          const uint8_t* token_mask, float* tv, float* kl, float* entropy,
                          int32_t* status, const dppo_opts* opts, void* cuda_stream);

/* Name of an error code (static string, never NULL). */
const char* dppo_error_string(int code);

/* Library version: major * 10000 + minor * 100 + patch. */
int dppo_version(void);

/* sizeof(dppo_opts) as this library was built: lets a binding written in another language check that its copy of the
 * struct has not drifted. */
size_t dppo_opts_size(void);

#ifdef __cplusplus
}
#endif
#endif /* DPPO_H_ */
