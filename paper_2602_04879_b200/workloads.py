"""Seeded synthetic inputs shaped like the paper's workloads.

These stand in for what a rollout engine and a trainer forward pass would hand
to the DPPO loss path: trainer logits, sampled token ids, the rollout policy's
stored log-probabilities (and optionally its top-K ids / probabilities),
per-token advantages and a token validity mask.  Nothing here evaluates the
method itself; the rollout-side softmax below is input generation (what the
inference engine stores), not part of the loss path.

Rows are generated in blocks from ``torch.Generator`` streams seeded by
(seed, block index), so any block of a large batch can be regenerated alone.
Generation runs on whichever device is asked for; CPU and CUDA streams differ,
which is fine because both sides of a comparison consume the same tensors.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

QWEN3_VOCAB = 151936          # vocabulary of the Qwen3 models the paper trains
BLOCK_ROWS = 512


@dataclasses.dataclass
class Batch:
    logits: Optional[torch.Tensor]          # [T, V] fp32 or bf16 (None for the LM-head workload)
    sampled_ids: torch.Tensor               # [T] int32
    mu_logp: torch.Tensor                   # [T] fp32, log mu(a_t)
    advantages: torch.Tensor                # [T] fp32
    token_mask: Optional[torch.Tensor]      # [T] uint8 or None (all valid)
    mu_topk_ids: Optional[torch.Tensor] = None   # [T, K] int32
    mu_topk_p: Optional[torch.Tensor] = None     # [T, K] fp32 probabilities
    hidden: Optional[torch.Tensor] = None        # [T, d] bf16 (LM-head workload)
    lm_head: Optional[torch.Tensor] = None       # [d, V] bf16
    meta: dict = dataclasses.field(default_factory=dict)

    @property
    def T(self):
        return int(self.sampled_ids.shape[0])


def _gen(device, seed, stream):
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(stream) * 7919 + 12345) % (2 ** 63 - 1))
    return g


def _rollout_side(mu_logits, K, g):
    """What the rollout engine stores for rows of rollout logits (fp32): a_t ~ softmax(mu) by
    Gumbel-max, log mu(a_t), and the top-K ids / probabilities of mu."""
    u = torch.rand(mu_logits.shape, generator=g, device=mu_logits.device, dtype=torch.float32)
    u = u.clamp_(1e-20, 1.0 - 1e-7)
    gumbel = -torch.log(-torch.log(u))
    a = torch.argmax(mu_logits + gumbel, dim=1)
    logp = torch.log_softmax(mu_logits, dim=1)
    mu_logp = logp.gather(1, a[:, None])[:, 0].contiguous()
    ids = ps = None
    if K > 0:
        top = torch.topk(logp, K, dim=1)
        ids = top.indices.to(torch.int32).contiguous()
        ps = torch.exp(top.values).contiguous()
    return a.to(torch.int32), mu_logp, ids, ps


def _zipf_offset(rows, V, g, device, exponent):
    """-exponent * ln(1 + rank) with a per-row affine permutation rank = (alpha*j + beta) mod V, alpha
    coprime to V, so that each row is peaked on its own tokens."""
    alpha = torch.randint(0, V, (rows,), generator=g, device=device, dtype=torch.int64)
    beta = torch.randint(0, V, (rows,), generator=g, device=device, dtype=torch.int64)
    alpha = alpha.cpu().tolist()
    fixed = []
    for x in alpha:
        x = max(1, x)
        while math.gcd(x, V) != 1:
            x += 1
        fixed.append(x % V if x % V else 1)
    alpha = torch.tensor(fixed, device=device, dtype=torch.int64)
    j = torch.arange(V, device=device, dtype=torch.int64)
    rank = (alpha[:, None] * j[None, :] + beta[:, None]) % V
    return -exponent * torch.log1p(rank.to(torch.float32))


def logits_rows(row0, rows, V, dtype, seed, device, sigma=3.0, zipf=1.1, peak=0.0, sigma_mu=0.1, K=0):
    """One block of rows: trainer logits (rounded to ``dtype``) and the rollout side built from
    (those rounded logits, upcast) + sigma_mu * N(0,1) in fp32."""
    assert row0 % BLOCK_ROWS == 0 or rows <= BLOCK_ROWS
    out_logits, out = [], []
    done = 0
    while done < rows:
        n = min(BLOCK_ROWS, rows - done)
        g = _gen(device, seed, (row0 + done) // BLOCK_ROWS)
        z = sigma * torch.randn((n, V), generator=g, device=device, dtype=torch.float32)
        if zipf:
            z += _zipf_offset(n, V, g, device, zipf)
        if peak:
            col = torch.randint(0, V, (n,), generator=g, device=device)
            z[torch.arange(n, device=device), col] += peak
        zq = z.to(dtype)
        mu_logits = zq.to(torch.float32) + sigma_mu * torch.randn((n, V), generator=g, device=device, dtype=torch.float32)
        out_logits.append(zq)
        out.append(_rollout_side(mu_logits, K, g))
        done += n
    logits = torch.cat(out_logits) if len(out_logits) > 1 else out_logits[0]
    a = torch.cat([o[0] for o in out])
    mu_logp = torch.cat([o[1] for o in out])
    ids = torch.cat([o[2] for o in out]) if K > 0 else None
    ps = torch.cat([o[3] for o in out]) if K > 0 else None
    return logits, a, mu_logp, ids, ps


def _group_advantages(n_resp, group, seed, kind):
    """Per-response advantages on the host: 'pm1' = +-1; 'group' = R - mean over the response group,
    R ~ Bernoulli(1/2), no division by the standard deviation (the paper's estimator)."""
    g = torch.Generator()
    g.manual_seed(int(seed) * 31 + 7)
    if kind == "pm1":
        return (torch.randint(0, 2, (n_resp,), generator=g).to(torch.float32) * 2 - 1)
    R = torch.randint(0, 2, (n_resp,), generator=g).to(torch.float32)
    R = R.view(-1, group)
    for i in range(R.shape[0]):           # a group with equal rewards carries no signal: flip one
        if R[i].min() == R[i].max():
            R[i, 0] = 1 - R[i, 0]
    return (R - R.mean(dim=1, keepdim=True)).reshape(-1)


def tiny_binary_tv(device="cpu", seed=0, T=256, V=4096, resp_len=16):
    """T tokens (responses of 16), fp32 logits ~ 2*N(0,1) with one entry per row boosted by +6,
    rollout noise 0.05, advantages +-1 per response, all valid."""
    logits, a, mu_logp, _, _ = logits_rows(0, T, V, torch.float32, seed, device, sigma=2.0, zipf=0.0, peak=6.0, sigma_mu=0.05)
    adv = _group_advantages(T // resp_len, 1, seed, "pm1").repeat_interleave(resp_len).to(device)
    return Batch(logits, a, mu_logp, adv, None, meta=dict(name="tiny_binary_tv", delta=0.2, variant="binary_tv"))


def qwen_vocab_rows(device, seed=1, n_resp=16, resp_len=1024, V=QWEN3_VOCAB, dtype=torch.bfloat16,
                    sigma_mu=0.1, K=0, group=16, row0=0, rows=None):
    """Rows of the Qwen3-vocabulary workloads: bf16 logits ~ 3*N(0,1) + Zipf(1.1) offset, rollout noise
    sigma_mu, group-mean-centred advantages constant within a response.  ``row0``/``rows`` select a
    slice of the n_resp*resp_len rows (row0 a multiple of the generator block)."""
    T = n_resp * resp_len
    rows = T - row0 if rows is None else rows
    logits, a, mu_logp, ids, ps = logits_rows(row0, rows, V, dtype, seed, device, sigma=3.0, zipf=1.1, sigma_mu=sigma_mu, K=K)
    adv = _group_advantages(n_resp, group, seed, "group").repeat_interleave(resp_len)[row0:row0 + rows].to(device)
    return Batch(logits, a, mu_logp, adv.contiguous(), None, ids, ps, meta=dict(name="qwen_vocab", K=K, T_total=T))


def ragged_lengths(n_resp=64, lo=128, hi=8192, seed=3):
    g = torch.Generator()
    g.manual_seed(int(seed) * 17 + 3)
    return torch.randint(lo, hi + 1, (n_resp,), generator=g).tolist()


def ragged_response(device, i, lengths, seed=3, max_len=8192, V=QWEN3_VOCAB, dtype=torch.bfloat16,
                    sigma_mu=0.3, K=64, group=8):
    """Response i of the ragged Top-K workload as one padded block of max_len rows with its token
    mask.  Padding rows hold zeros everywhere (ids 0, log-prob 0)."""
    L = int(lengths[i])
    logits = torch.zeros((max_len, V), dtype=dtype, device=device)
    a = torch.zeros(max_len, dtype=torch.int32, device=device)
    mu_logp = torch.zeros(max_len, dtype=torch.float32, device=device)
    ids = torch.zeros((max_len, K), dtype=torch.int32, device=device)
    ps = torch.zeros((max_len, K), dtype=torch.float32, device=device)
    lg, aa, ml, ii, pp = logits_rows(0, L, V, dtype, seed * 1009 + i, device, sigma=3.0, zipf=1.1, sigma_mu=sigma_mu, K=K)
    logits[:L], a[:L], mu_logp[:L], ids[:L], ps[:L] = lg, aa, ml, ii, pp
    adv_resp = _group_advantages(len(lengths), group, seed, "group")
    adv = torch.full((max_len,), float(adv_resp[i]), dtype=torch.float32, device=device)
    mask = torch.zeros(max_len, dtype=torch.uint8, device=device)
    mask[:L] = 1
    return Batch(logits, a, mu_logp, adv, mask, ids, ps, meta=dict(name="ragged_topk_kl", K=K, length=L,
                                                                   n_valid_total=int(sum(lengths))))


def lm_head_workload(device, seed=5, T=8192, d=2048, V=QWEN3_VOCAB, resp_len=512, sigma_w=0.02, sigma_mu=0.1, K=0):
    """hidden [T,d] bf16 ~ N(0,1), LM head W [d,V] bf16 ~ sigma_w*N(0,1); the rollout side is built from
    hidden x W (fp32 accumulation, computed here only to generate inputs) + sigma_mu*N(0,1)."""
    g = _gen(device, seed, 0)
    H = torch.randn((T, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    W = (sigma_w * torch.randn((d, V), generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)
    a_l, ml_l, id_l, p_l = [], [], [], []
    Wf = W.to(torch.float32) if device == "cpu" or str(device) == "cpu" else None
    for r0 in range(0, T, BLOCK_ROWS):
        n = min(BLOCK_ROWS, T - r0)
        gb = _gen(device, seed, 1 + r0 // BLOCK_ROWS)
        if Wf is not None:
            z = H[r0:r0 + n].to(torch.float32) @ Wf
        else:
            z = (H[r0:r0 + n] @ W).to(torch.float32)
        z = z + sigma_mu * torch.randn((n, V), generator=gb, device=device, dtype=torch.float32)
        a, ml, ids, ps = _rollout_side(z, K, gb)
        a_l.append(a)
        ml_l.append(ml)
        id_l.append(ids)
        p_l.append(ps)
    adv = _group_advantages(max(1, T // resp_len), 1, seed, "pm1").repeat_interleave(resp_len)[:T].to(device)
    if adv.shape[0] < T:
        adv = torch.cat([adv, adv.new_ones(T - adv.shape[0])])
    return Batch(None, torch.cat(a_l), torch.cat(ml_l), adv.contiguous(), None,
                 torch.cat(id_l) if K > 0 else None, torch.cat(p_l) if K > 0 else None, hidden=H, lm_head=W,
                 meta=dict(name="lm_head_binary_tv", delta=0.2, K=K))
