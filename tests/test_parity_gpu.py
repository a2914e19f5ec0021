"""GPU-vs-oracle parity through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import paper_2602_04879_b200 as dppo
from paper_2602_04879_b200 import workloads as wl
from oracle import dppo_oracle as O

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KERNELS = {"ring": dppo.KERNEL_RING, "generic": dppo.KERNEL_GENERIC}


def _run(batch, variant, K, delta, kernel, dlogits_f32=False, loss_scale=0.0, want_stats=True, dlogits=None, is_cap=0.0, eps_low=0.0,
         row_cluster=0):
    out = dppo.dppo_loss_fwd_bwd(batch.logits, batch.sampled_ids, batch.mu_logp, batch.advantages, batch.token_mask,
                                 variant, K, delta, batch.mu_topk_ids, batch.mu_topk_p, loss_scale=loss_scale,
                                 dlogits_f32=dlogits_f32, kernel=kernel, want_stats=want_stats, dlogits=dlogits,
                                 is_cap=is_cap, eps_low=eps_low, row_cluster=row_cluster)
    torch.cuda.synchronize()
    return out


def _stress_delta(D):
    """A threshold near the median divergence that sits in the widest nearby gap between two rows'
    values, so that no row is within the exemption band of it."""
    d = np.sort(D.detach().cpu().numpy().astype(np.float64))
    d = d[np.isfinite(d) & (d > 0)]
    k = len(d) // 2
    lo, hi = max(0, k - 8), min(len(d) - 1, k + 8)
    gaps = d[lo + 1:hi + 1] - d[lo:hi]
    i = int(np.argmax(gaps)) + lo
    assert gaps.max() > 2.5e-6
    return float(np.float32(0.5 * (d[i] + d[i + 1])))


def _full_check(batch, variant, K, delta, kernel, dlogits_f32=False, loss_scale=0.0, expect_blocked=None, is_cap=0.0, eps_low=0.0,
                row_cluster=0):
    out = _run(batch, variant, K, delta, kernel, dlogits_f32, loss_scale, is_cap=is_cap, eps_low=eps_low, row_cluster=row_cluster)
    assert int(out["status"].item()) == 0
    h = P.host_inputs(batch)
    ora = P.run_oracle(h, variant, K, delta, None if loss_scale == 0.0 else loss_scale, is_cap=is_cap if is_cap > 0 else None,
                       eps_low=eps_low if eps_low > 0 else None)
    n_exempt, d_err = P.check_scalars(out["divergence"].cpu().numpy(), out["mask"].cpu().numpy(), ora, h, delta,
                                      eps_low=eps_low if eps_low > 0 else None)
    bf16_in = batch.logits.dtype == torch.bfloat16
    info = P.check_loss(float(out["loss"].item()), ora["loss"], bf16_in, ora["row_loss"])
    dinfo = P.check_dlogits(out["dlogits"], ora["dlogits"], out_is_bf16=(bf16_in and not dlogits_f32))
    valid = np.ones(batch.T, bool) if h["token_mask"] is None else h["token_mask"] != 0
    blocked = int(((ora["M"] == 0) & valid).sum())
    if expect_blocked is not None:
        assert expect_blocked(blocked, int(valid.sum())), f"blocked {blocked} of {int(valid.sum())}"
    st = out["stats"].cpu().numpy()
    assert st[0] == valid.sum() and st[1] == blocked
    assert abs(st[4] - np.sum(np.abs(np.exp(h["mu_logp"][valid]) - ora["r"][valid] * np.exp(h["mu_logp"][valid])))) <= 1e-3 * max(1.0, st[4])
    return out, ora, dict(n_exempt=n_exempt, d_err=d_err, **info, **dinfo)


def _grad_scale(batch, scale, ora, rows):
    """max |dlogits| over the WHOLE tensor, for the tolerance of a check on sampled rows, without looking at the GPU's
    output: every entry obeys |dlogits_tj| <= s |A_t| r_t max(pi_tj, 1 - pi_t(a)) <= s |A_t| r_t, so the maximum over all
    rows lies between the largest entry of the sampled oracle rows and s max_t |A_t| r_t; the smaller (stricter) of the
    two, the oracle's own maximum over the sampled rows, is the denominator."""
    upper = float(scale) * float(batch.advantages.abs().max().item()) * float(np.max(ora["r"]))
    mx = float(np.abs(ora["dlogits"]).max())
    assert 0 < mx <= upper * (1 + 1e-12) or upper == 0
    return mx


# ------------------------------------------------------------------------------------- config 1

@pytest.mark.parametrize("kernel", sorted(KERNELS))
def test_tiny_binary_tv_fp32(kernel):
    """T=256, V=4096, fp32 logits, Binary-TV, delta=0.2, all valid, seed 0."""
    b = wl.tiny_binary_tv(DEV, seed=0)
    _full_check(b, dppo.BINARY_TV, 0, 0.2, KERNELS[kernel])
    # mask-stress: threshold at the median divergence so that a good share of rows is blocked
    out = _run(b, dppo.BINARY_TV, 0, 0.2, KERNELS[kernel])
    med = _stress_delta(out["divergence"])
    _full_check(b, dppo.BINARY_TV, 0, med, KERNELS[kernel], expect_blocked=lambda k, n: 0.1 * n < k < 0.5 * n)
    _full_check(b, dppo.BINARY_KL, 0, 1e-4, KERNELS[kernel])


# ------------------------------------------------------------------------------------- config 2

@pytest.fixture(scope="module")
def qwen_rows():
    """333 rows of the Qwen3-vocabulary workload (bf16, V=151936) with top-64 lists; 333 rows on 148 SMs
    give two full waves and a ragged third; a row is 38 chunks of 8 KB with a 768-byte tail."""
    return wl.qwen_vocab_rows(DEV, seed=1, n_resp=9, resp_len=37, K=64, group=9)


@pytest.mark.parametrize("variant,delta", [(dppo.BINARY_TV, 0.1), (dppo.BINARY_TV, 0.2), (dppo.BINARY_KL, 0.1), (dppo.BINARY_KL, 0.2)])
def test_qwen_binary(qwen_rows, variant, delta):
    out, ora, info = _full_check(qwen_rows, variant, 0, delta, dppo.KERNEL_RING)
    assert info["frac_literal"] > 0.999999


@pytest.mark.parametrize("variant", [dppo.BINARY_TV, dppo.BINARY_KL])
def test_qwen_binary_mask_stress(qwen_rows, variant):
    out = _run(qwen_rows, variant, 0, 1.0, dppo.KERNEL_RING)
    med = _stress_delta(out["divergence"])
    _full_check(qwen_rows, variant, 0, med, dppo.KERNEL_RING, expect_blocked=lambda k, n: 0.1 * n < k < 0.5 * n)


def test_qwen_fp32_gradient_and_generic_kernel(qwen_rows):
    """fp32 gradient output meets the literal 2e-3*max bound; the scalar kernel agrees with the oracle too."""
    _, _, info = _full_check(qwen_rows, dppo.BINARY_TV, 0, 0.02, dppo.KERNEL_RING, dlogits_f32=True)
    assert info["max_err_over_max"] < 2e-5
    _full_check(qwen_rows, dppo.BINARY_TV, 0, 0.02, dppo.KERNEL_GENERIC)
    _full_check(qwen_rows, dppo.TOPK_KL, 64, 0.02, dppo.KERNEL_GENERIC, dlogits_f32=True)


@pytest.mark.parametrize("kernel", sorted(KERNELS))
def test_truncated_importance_weight_and_ppo_clip_baseline(kernel, qwen_rows):
    """min(r, C) of Eq. unified_grad, the unmasked PG-IS / CISPO baselines (delta = inf) and the PPO ratio-clip mask."""
    b = wl.Batch(qwen_rows.logits, qwen_rows.sampled_ids, qwen_rows.mu_logp, qwen_rows.advantages, None)
    base = _run(b, dppo.BINARY_TV, 0, 1.0, KERNELS[kernel])
    h = P.host_inputs(b)
    r = P.run_oracle(h, O.BINARY_TV, 0, 1.0, None, want_grad=False)["r"]
    C = float(np.float32(np.median(r)))                      # about half of the rows are truncated
    _, ora, _ = _full_check(b, dppo.BINARY_TV, 0, 0.02, KERNELS[kernel], is_cap=C)
    assert 0.3 < np.mean(ora["r"] > C) < 0.7
    out, ora, _ = _full_check(b, dppo.BINARY_KL, 0, float("inf"), KERNELS[kernel], is_cap=3.0)     # CISPO / PG-TIS
    assert np.all(ora["M"] == 1)
    # PPO / GRPO clip with the paper's ranges: few rows clipped at noise 0.1; a tight range clips a good share
    _full_check(b, dppo.PPO_CLIP, 0, 0.28, KERNELS[kernel], eps_low=0.2)
    rr = np.sort(np.abs(r - 1.0))
    eh = float(np.float32(0.5 * (rr[len(rr) // 2] + rr[len(rr) // 2 + 1])))
    el = float(np.float32(0.5 * (rr[len(rr) // 3] + rr[len(rr) // 3 + 1])))
    _full_check(b, dppo.PPO_CLIP, 0, eh, KERNELS[kernel], eps_low=el, expect_blocked=lambda k, n: 0.1 * n < k < 0.5 * n)
    # minimal mask of Sec. 5.3 (signed D = mu(a) - pi(a); only negative samples are ever blocked)
    dd = np.exp(h["mu_logp"]) - r * np.exp(h["mu_logp"])
    pos = np.sort(dd[(dd > 0) & (h["advantages"] < 0)])
    dm = float(np.float32(0.5 * (pos[len(pos) // 2] + pos[len(pos) // 2 + 1])))
    out, ora, _ = _full_check(b, dppo.MINIMAL_MASK, 0, dm, KERNELS[kernel], expect_blocked=lambda k, n: 0 < k < 0.5 * n)
    assert np.all(h["advantages"][ora["M"] == 0] < 0)


# ------------------------------------------------------------------------------------- config 3

def test_qwen_topk_tv_k20(qwen_rows):
    b = qwen_rows
    b20 = wl.Batch(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None,
                   b.mu_topk_ids[:, :20].contiguous(), b.mu_topk_p[:, :20].contiguous())
    _full_check(b20, dppo.TOPK_TV, 20, 0.2, dppo.KERNEL_RING)
    out = _run(b20, dppo.TOPK_TV, 20, 1.0, dppo.KERNEL_RING)
    med = _stress_delta(out["divergence"])
    _full_check(b20, dppo.TOPK_TV, 20, med, dppo.KERNEL_RING, expect_blocked=lambda k, n: 0.1 * n < k < 0.5 * n)
    # Top-K refines Binary: D_bin <= D_topk row by row (App. B)
    bin_ = _run(b20, dppo.BINARY_TV, 0, 1.0, dppo.KERNEL_RING)
    assert torch.all(bin_["divergence"] <= out["divergence"] + 1e-6)


@pytest.mark.parametrize("V,n_resp,resp_len", [(32000, 15, 40), (128256, 10, 31), (262144, 5, 31), (1 << 20, 3, 13)])
def test_other_vocabulary_sizes(V, n_resp, resp_len):
    """Vocabularies of other model families and a one-million-entry one (32 and 128 chunks of 16 KB per row: the first read then
    leads the second by one row and two chunks instead of the usual margin), bf16, rows on a ragged last wave: Top-K KL and
    Binary-TV with a threshold that blocks part of the rows, every output against the oracle."""
    b = wl.qwen_vocab_rows(DEV, seed=11, n_resp=n_resp, resp_len=resp_len, V=V, K=20, group=n_resp, sigma_mu=0.2)
    out = _run(b, dppo.TOPK_KL, 20, 1e9, dppo.KERNEL_AUTO)
    _full_check(b, dppo.TOPK_KL, 20, _stress_delta(out["divergence"]), dppo.KERNEL_AUTO, expect_blocked=lambda k, n: 0.05 * n < k < 0.5 * n)
    bb = wl.Batch(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, None, None)
    out = _run(bb, dppo.BINARY_TV, 0, 1.0, dppo.KERNEL_AUTO)
    _full_check(bb, dppo.BINARY_TV, 0, _stress_delta(out["divergence"]), dppo.KERNEL_AUTO, expect_blocked=lambda k, n: 0.05 * n < k < 0.5 * n)


@pytest.mark.parametrize("row_cluster", [2, 4])
def test_rows_shared_by_the_sms_of_a_cluster(row_cluster):
    """``opts.row_cluster`` forced on shapes the automatic choice would give one SM per row: 2 or 4 SMs stream alternate
    chunks of a row and exchange their partial sums.  Rows of 19 chunks with a ragged tail (the chunks do not divide evenly),
    invalid rows (zero fill split among the SMs), shifted rows, rows of a single chunk (SMs without any chunk of the row),
    fewer rows than clusters; every output against the oracle, and twice the same bits."""
    b = wl.qwen_vocab_rows(DEV, seed=13, n_resp=5, resp_len=31, K=20, group=5, sigma_mu=0.2)
    b.token_mask = (torch.arange(b.T, device=DEV) % 11 != 3).to(torch.uint8)
    b.logits[3] = float("nan")                                  # an invalid row's content must not matter
    out = _run(b, dppo.TOPK_KL, 20, 1e9, dppo.KERNEL_RING, row_cluster=row_cluster)
    o1, _, _ = _full_check(b, dppo.TOPK_KL, 20, _stress_delta(out["divergence"][b.token_mask != 0]), dppo.KERNEL_RING, row_cluster=row_cluster,
                           expect_blocked=lambda k, n: 0.05 * n < k < 0.5 * n)
    o2 = _run(b, dppo.TOPK_KL, 20, _stress_delta(out["divergence"][b.token_mask != 0]), dppo.KERNEL_RING, row_cluster=row_cluster)
    assert torch.equal(o1["dlogits"], o2["dlogits"]) and torch.equal(o1["loss"], o2["loss"]) and torch.equal(o1["divergence"], o2["divergence"])
    _full_check(b, dppo.BINARY_KL, 0, 0.001, dppo.KERNEL_RING, row_cluster=row_cluster)
    # one SM per row gives the same mask and divergence up to the order of the additions in the row sums
    ref = _run(b, dppo.BINARY_KL, 0, 0.001, dppo.KERNEL_RING, row_cluster=1)
    got = _run(b, dppo.BINARY_KL, 0, 0.001, dppo.KERNEL_RING, row_cluster=row_cluster)
    assert torch.allclose(ref["divergence"], got["divergence"], atol=2e-6, rtol=1e-5)
    # shifted rows (a vocabulary that is not a multiple of 8), several chunks, Top-K, invalid rows
    T, V = 150, 40003
    logits, a, mu_logp, ids, ps = wl.logits_rows(0, T, V, torch.bfloat16, 23, DEV, sigma=2.0, zipf=1.1, sigma_mu=0.5, K=5)
    adv = torch.where(torch.arange(T, device=DEV) % 3 == 0, -1.0, 0.7).to(torch.float32)
    tok = (torch.arange(T, device=DEV) % 7 != 2).to(torch.uint8)
    bs = wl.Batch(logits, a, mu_logp, adv, tok, ids, ps)
    _full_check(bs, dppo.TOPK_TV, 5, 0.01, dppo.KERNEL_RING, row_cluster=row_cluster)
    # rows of one chunk, fp32, and fewer rows than clusters
    _full_check(wl.tiny_binary_tv(DEV, seed=0), dppo.BINARY_TV, 0, 0.2, dppo.KERNEL_RING, row_cluster=row_cluster)
    _full_check(wl.tiny_binary_tv(DEV, seed=2, T=3, V=4096, resp_len=1), dppo.BINARY_TV, 0, 0.01, dppo.KERNEL_RING, row_cluster=row_cluster)


# ------------------------------------------------------------------------------------- config 4

def test_ragged_topk_kl_k64():
    """Ragged responses in padded blocks with a token mask, TopK-KL K=64, delta=0.05, rollout noise 0.3;
    each padded block is one call with the global token-mean scale, as the full-size workload is run."""
    lengths = [37, 128, 5, 90]
    max_len = 128
    n_valid = sum(lengths)
    scale = 1.0 / n_valid
    total_gpu, total_ora, blocked = 0.0, 0.0, 0
    for i in range(len(lengths)):
        b = wl.ragged_response(DEV, i, lengths, seed=3, max_len=max_len, K=64, group=4)
        # poison the padding so that a kernel reading it would be caught
        b.logits[lengths[i]:] = float("nan")
        b.sampled_ids[lengths[i]:] = -7
        out, ora, info = _full_check(b, dppo.TOPK_KL, 64, 0.05, dppo.KERNEL_RING, loss_scale=scale)
        total_gpu += float(out["loss"].item())
        total_ora += ora["loss"]
        blocked += int((ora["M"][: lengths[i]] == 0).sum())
        assert not out["dlogits"][lengths[i]:].any() and not out["divergence"][lengths[i]:].any()
    assert blocked > 0
    assert abs(total_gpu - total_ora) <= 1e-3 * abs(total_ora)


# ------------------------------------------------------------------------------------- edge cases

@pytest.mark.parametrize("kernel", sorted(KERNELS))
@pytest.mark.parametrize("V,dtype", [(8, torch.bfloat16), (4104, torch.bfloat16), (4, torch.float32), (2052, torch.float32)])
def test_small_vocab_topk_full(kernel, V, dtype):
    """K = V (exact divergence, empty 'other' bucket) and K = 0 (Binary) on small vocabularies."""
    T = 40
    logits, a, mu_logp, ids, ps = wl.logits_rows(0, T, V, dtype, 11, DEV, sigma=2.0, zipf=1.1, sigma_mu=0.5, K=V)
    adv = torch.where(torch.arange(T, device=DEV) % 3 == 0, -1.0, 0.7).to(torch.float32)
    adv[5] = 0.0
    tok = torch.ones(T, dtype=torch.uint8, device=DEV)
    tok[7] = 0
    b = wl.Batch(logits, a, mu_logp, adv, tok, ids, ps)
    for variant in (dppo.TOPK_TV, dppo.TOPK_KL):
        _full_check(b, variant, V, 0.05, KERNELS[kernel])
        b0 = wl.Batch(logits, a, mu_logp, adv, tok, None, None)
        o_top0, _, _ = _full_check(b0, variant, 0, 0.05, KERNELS[kernel])
        o_bin, _, _ = _full_check(b0, variant - 2, 0, 0.05, KERNELS[kernel])
        assert torch.allclose(o_top0["divergence"], o_bin["divergence"], atol=1e-6)


def test_odd_vocab_and_strided_rows():
    T, V = 19, 1001
    logits, a, mu_logp, ids, ps = wl.logits_rows(0, T, V, torch.bfloat16, 12, DEV, sigma=2.0, zipf=1.1, sigma_mu=0.5, K=7)
    adv = torch.linspace(-1, 1, T, device=DEV)
    b = wl.Batch(logits, a, mu_logp, adv, None, ids, ps)
    # contiguous rows of an odd length: row starts are only element aligned; the bulk-copy kernel takes them as
    # "shifted" rows when logits and dlogits are shifted alike, the scalar kernel takes everything
    for kernel in (dppo.KERNEL_AUTO, dppo.KERNEL_RING, dppo.KERNEL_GENERIC):
        _full_check(b, dppo.TOPK_KL, 7, 0.01, kernel)
    # fp32 gradient of bf16 logits of odd length: the two tensors cannot be shifted alike
    with pytest.raises(dppo.DppoError) as e:
        _run(b, dppo.TOPK_KL, 7, 0.01, dppo.KERNEL_RING, dlogits_f32=True)
    assert "alignment" in str(e.value)
    _full_check(b, dppo.TOPK_KL, 7, 0.01, dppo.KERNEL_AUTO, dlogits_f32=True)
    # strided rows (a view into a wider buffer)
    wide = torch.zeros((T, V + 23), dtype=torch.bfloat16, device=DEV)
    wide[:, :V] = logits
    b2 = wl.Batch(wide[:, :V], a, mu_logp, adv, None, ids, ps)
    _full_check(b2, dppo.TOPK_TV, 7, 0.01, dppo.KERNEL_AUTO)


@pytest.mark.parametrize("T,V,dtype", [(333, 20011, torch.bfloat16), (200, 5003, torch.float32), (40, 8193, torch.bfloat16),
                                       (7, 3, torch.float32), (150, 16385, torch.bfloat16)])
def test_shifted_rows_through_the_bulk_copy_kernel(T, V, dtype):
    """Vocabularies that are not a multiple of 8 (bf16) / 4 (fp32) elements, contiguous: every row starts at another offset
    from a 16-byte boundary.  Several chunks per row, several rows per CTA, invalid rows (zero fill), Top-K, in place."""
    K = min(5, V)
    logits, a, mu_logp, ids, ps = wl.logits_rows(0, T, V, dtype, 21, DEV, sigma=2.0, zipf=1.1, sigma_mu=0.5, K=K)
    adv = torch.where(torch.arange(T, device=DEV) % 3 == 0, -1.0, 0.7).to(torch.float32)
    tok = (torch.arange(T, device=DEV) % 7 != 2).to(torch.uint8)
    b = wl.Batch(logits, a, mu_logp, adv, tok, ids, ps)
    out, ora, _ = _full_check(b, dppo.BINARY_TV, 0, 0.05, dppo.KERNEL_RING)
    _full_check(b, dppo.TOPK_TV, K, 0.01, dppo.KERNEL_RING)
    gen = _run(b, dppo.BINARY_TV, 0, 0.05, dppo.KERNEL_GENERIC)
    assert torch.equal(gen["mask"], out["mask"])
    # in place: the gradient overwrites the logits
    z = logits.clone()
    bi = wl.Batch(z, a, mu_logp, adv, tok, ids, ps)
    inpl = _run(bi, dppo.BINARY_TV, 0, 0.05, dppo.KERNEL_RING, dlogits=z)
    torch.cuda.synchronize()
    assert torch.equal(inpl["dlogits"], out["dlogits"]) and inpl["dlogits"].data_ptr() == z.data_ptr()
    # guard bytes around the output stay untouched (edge vectors are written element by element)
    pad = torch.full((T * V + 64,), 7.0, dtype=dtype, device=DEV)
    view = pad[32:32 + T * V].view(T, V)          # 32 elements in: 16-byte aligned base for both element sizes
    _run(b, dppo.BINARY_TV, 0, 0.05, dppo.KERNEL_RING, dlogits=view)
    torch.cuda.synchronize()
    assert torch.equal(view, out["dlogits"]) and torch.all(pad[:32] == 7.0) and torch.all(pad[32 + T * V:] == 7.0)


def test_empty_and_fully_masked():
    V = 4096
    b = wl.tiny_binary_tv(DEV, seed=2, T=32, V=V)
    empty = wl.Batch(b.logits[:0], b.sampled_ids[:0], b.mu_logp[:0], b.advantages[:0], None)
    out = _run(empty, dppo.BINARY_TV, 0, 0.2, dppo.KERNEL_AUTO, want_stats=False)
    assert float(out["loss"].item()) == 0.0 and out["dlogits"].shape == (0, V)
    b.token_mask = torch.zeros(32, dtype=torch.uint8, device=DEV)
    for k in KERNELS.values():
        out = _run(b, dppo.BINARY_TV, 0, 0.2, k)
        assert float(out["loss"].item()) == 0.0 and not out["dlogits"].any() and not out["mask"].any()
        assert out["stats"][0].item() == 0


@pytest.mark.parametrize("kernel", sorted(KERNELS))
def test_in_place_and_determinism(kernel, qwen_rows):
    b = qwen_rows
    ref = _run(b, dppo.BINARY_KL, 0, 0.01, KERNELS[kernel])
    again = _run(b, dppo.BINARY_KL, 0, 0.01, KERNELS[kernel])
    assert torch.equal(ref["dlogits"], again["dlogits"]) and torch.equal(ref["loss"], again["loss"])
    buf = b.logits.clone()
    inpl = wl.Batch(buf, b.sampled_ids, b.mu_logp, b.advantages, None)
    out = _run(inpl, dppo.BINARY_KL, 0, 0.01, KERNELS[kernel], dlogits=buf)
    assert torch.equal(out["dlogits"], ref["dlogits"]) and torch.equal(out["divergence"], ref["divergence"])


@pytest.mark.parametrize("kernel", sorted(KERNELS))
def test_device_detected_anomalies_set_status(kernel):
    """Bad ids and non-finite rows never trap: status bits are set and the row is treated as invalid."""
    b = wl.tiny_binary_tv(DEV, seed=4, T=64, V=4096)
    _, _, _, ids, ps = wl.logits_rows(0, 64, 4096, torch.float32, 4, DEV, sigma=2.0, zipf=0.0, peak=6.0, sigma_mu=0.05, K=5)
    b.mu_topk_ids, b.mu_topk_p = ids.clone(), ps
    b.sampled_ids[3] = 4096
    b.sampled_ids[9] = -1
    b.mu_topk_ids[11, 2] = 1 << 20
    b.logits[17, 100] = float("nan")
    b.logits[21, 5] = float("inf")
    b.logits[30, :] = float("-inf")
    out = _run(b, dppo.TOPK_KL, 5, 0.05, KERNELS[kernel])
    assert int(out["status"].item()) == (dppo.binding.STATUS_BAD_SAMPLED_ID | dppo.binding.STATUS_BAD_TOPK_ID | dppo.binding.STATUS_NONFINITE_ROW)
    bad = [3, 9, 11, 17, 21, 30]
    for t in bad:
        assert not out["dlogits"][t].any() and out["mask"][t].item() == 0 and out["divergence"][t].item() == 0
    good = [t for t in range(64) if t not in bad]
    h = P.host_inputs(b, good)
    ora = P.run_oracle(h, O.TOPK_KL, 5, 0.05, 1.0 / 64)
    P.check_scalars(out["divergence"][good].cpu().numpy(), out["mask"][good].cpu().numpy(), ora, h, 0.05)
    P.check_dlogits(out["dlogits"][good], ora["dlogits"], out_is_bf16=False)
    # -inf entries in an otherwise finite row are fine (zero probability)
    b2 = wl.tiny_binary_tv(DEV, seed=5, T=16, V=4096)
    b2.logits[:, 7::13] = float("-inf")
    b2.sampled_ids[:] = 8
    _full_check(b2, dppo.BINARY_TV, 0, 0.2, KERNELS[kernel])


# ------------------------------------------------------------------------------------- host-buffer entry point

def test_host_buffer_entry_matches_device_entry(qwen_rows):
    b = qwen_rows
    dev = _run(b, dppo.TOPK_TV, 64, 0.02, dppo.KERNEL_AUTO)
    pin = lambda x: x.cpu().pin_memory()
    out = dppo.dppo_loss_fwd_bwd_host(pin(b.logits), pin(b.sampled_ids), pin(b.mu_logp), pin(b.advantages), None,
                                      dppo.TOPK_TV, 64, 0.02, pin(b.mu_topk_ids), pin(b.mu_topk_p),
                                      rows_per_chunk=100, want_dlogits=True, device=DEV)
    assert out["status"] == 0
    assert torch.equal(out["divergence"], dev["divergence"].cpu()) and torch.equal(out["mask"], dev["mask"].cpu())
    # same kernels on the same rows; only the scale differs in its last fp32 bit, which may move an
    # occasional gradient entry to the neighbouring bf16 value
    a_, b_ = out["dlogits"].float(), dev["dlogits"].cpu().float()
    assert torch.all((a_ - b_).abs() <= 2.0 ** -7 * b_.abs()) and (a_ != b_).float().mean() < 1e-2
    # the host entry passes the token-mean scale as an fp32 argument and adds the chunks' partial losses
    assert abs(out["loss"] - float(dev["loss"].item())) <= 1e-4 * abs(out["loss"]) + 1e-12


# ------------------------------------------------------------------------------------- full size

def test_full_size_binary_tv_sampled_rows():
    """The benchmark's configuration (T=16384, V=151936, bf16, Binary-TV, delta=0.2): mask, divergence and
    loss against the oracle on all rows (forward only), the gradient on sampled rows, and properties that
    hold at any size."""
    T = 16384
    b = wl.qwen_vocab_rows(DEV, seed=1)
    assert b.T == T
    out = _run(b, dppo.BINARY_TV, 0, 0.2, dppo.KERNEL_AUTO)
    assert int(out["status"].item()) == 0
    rng = np.random.default_rng(0)
    rows = np.sort(rng.choice(T, 48, replace=False))
    h = P.host_inputs(b, rows)
    ora = P.run_oracle(h, O.BINARY_TV, 0, 0.2, 1.0 / T)
    P.check_scalars(out["divergence"].cpu().numpy()[rows], out["mask"].cpu().numpy()[rows], ora, h, 0.2)
    mx = _grad_scale(b, 1.0 / T, ora, rows)
    P.check_dlogits(out["dlogits"][torch.as_tensor(rows, device=DEV)], ora["dlogits"], out_is_bf16=True, max_abs=mx)
    # the loss over a random eighth of the rows (token mask), same tensors, oracle forward only
    tok = (torch.rand(T, generator=torch.Generator().manual_seed(5)) < 0.125).to(torch.uint8)
    idx = np.nonzero(tok.numpy())[0]
    bm = wl.Batch(b.logits, b.sampled_ids, b.mu_logp, b.advantages, tok.to(DEV))
    outm = _run(bm, dppo.BINARY_TV, 0, 0.2, dppo.KERNEL_AUTO)
    hb = P.host_inputs(bm, idx)
    hb["token_mask"] = None
    ob = P.run_oracle(hb, O.BINARY_TV, 0, 0.2, 1.0 / len(idx), want_grad=False)
    P.check_scalars(outm["divergence"].cpu().numpy()[idx], outm["mask"].cpu().numpy()[idx], ob, hb, 0.2)
    P.check_loss(float(outm["loss"].item()), ob["loss"], True, ob["row_loss"])
    assert outm["stats"][0].item() == len(idx)
    inv = torch.nonzero(tok == 0)[:, 0][:64].to(DEV)
    assert not outm["dlogits"][inv].any()
    # valid rows of the masked call equal the unmasked call's rows up to the scale factor T/len(idx)
    t0 = int(idx[0])
    ratio = (outm["dlogits"][t0].float() / out["dlogits"][t0].float().clamp_min(1e-30))[out["dlogits"][t0].float() > 1e-20]
    assert torch.allclose(ratio, torch.full_like(ratio, T / len(idx)), rtol=2e-2)
    # properties: gradient rows sum to ~0 (bf16 rounding noise), blocked rows are exactly zero
    sums = out["dlogits"].to(torch.float32).sum(dim=1).abs().max().item()
    assert sums <= 2e-3 * float(np.abs(ora["dlogits"]).max()) * 40
    blocked = torch.nonzero(out["mask"] == 0)[:, 0]
    assert not out["dlogits"][blocked].any()


def test_full_size_topk_tv_k20_sampled_rows():
    """Config 3 at full size (T=16384, V=151936, bf16, TopK-TV, K=20, delta=0.2): sampled rows against the oracle."""
    T = 16384
    b = wl.qwen_vocab_rows(DEV, seed=1, K=20)
    out = _run(b, dppo.TOPK_TV, 20, 0.2, dppo.KERNEL_AUTO)
    assert int(out["status"].item()) == 0
    rows = np.sort(np.random.default_rng(3).choice(T, 40, replace=False))
    h = P.host_inputs(b, rows)
    ora = P.run_oracle(h, O.TOPK_TV, 20, 0.2, 1.0 / T)
    P.check_scalars(out["divergence"].cpu().numpy()[rows], out["mask"].cpu().numpy()[rows], ora, h, 0.2)
    mx = _grad_scale(b, 1.0 / T, ora, rows)
    P.check_dlogits(out["dlogits"][torch.as_tensor(rows, device=DEV)], ora["dlogits"], out_is_bf16=True, max_abs=mx)
    # stress threshold on the same tensors: the mask of the sampled rows still agrees
    d_all = out["divergence"]
    delta = _stress_delta(d_all[torch.as_tensor(rows, device=DEV)])
    out2 = _run(b, dppo.TOPK_TV, 20, delta, dppo.KERNEL_AUTO)
    ora2 = P.run_oracle(h, O.TOPK_TV, 20, delta, 1.0 / T, want_grad=False)
    P.check_scalars(out2["divergence"].cpu().numpy()[rows], out2["mask"].cpu().numpy()[rows], ora2, h, delta)
    assert 0 < int((ora2["M"] == 0).sum()) < len(rows)


def test_full_size_ragged_topk_kl_k64_one_response():
    """Config 4, one padded response block at full size (8192 rows x V=151936, K=64, rollout noise 0.3, delta=0.05),
    with the global token-mean scale of the 64-response batch, as the whole batch would be streamed."""
    lengths = wl.ragged_lengths()
    n_valid = int(sum(lengths))
    i = 7                                          # a response of medium length
    L = int(lengths[i])
    b = wl.ragged_response(DEV, i, lengths)
    b.logits[L:] = float("nan")                    # a kernel that read the padding would be caught
    out = _run(b, dppo.TOPK_KL, 64, 0.05, dppo.KERNEL_AUTO, loss_scale=1.0 / n_valid)
    assert int(out["status"].item()) == 0 and out["stats"][0].item() == L
    rows = np.sort(np.random.default_rng(4).choice(L, 40, replace=False))
    h = P.host_inputs(b, rows)
    h["token_mask"] = None
    ora = P.run_oracle(h, O.TOPK_KL, 64, 0.05, 1.0 / n_valid)
    P.check_scalars(out["divergence"].cpu().numpy()[rows], out["mask"].cpu().numpy()[rows], ora, h, 0.05)
    assert 0 < int((ora["M"] == 0).sum())          # this workload does leave the trust region
    mx = _grad_scale(b, 1.0 / n_valid, ora, rows)
    P.check_dlogits(out["dlogits"][torch.as_tensor(rows, device=DEV)], ora["dlogits"], out_is_bf16=True, max_abs=mx)
    assert not out["dlogits"][L:].any() and not out["mask"][L:].any() and not out["divergence"][L:].any()


def test_host_buffer_entry_with_an_odd_vocabulary():
    """Host buffers whose rows are only element aligned: the staged chunks are contiguous, so they take the shifted-row path."""
    T, V = 230, 20011
    logits, a, mu_logp, ids, ps = wl.logits_rows(0, T, V, torch.bfloat16, 31, DEV, sigma=2.0, zipf=1.1, sigma_mu=0.5, K=0)
    adv = torch.where(torch.arange(T, device=DEV) % 2 == 0, -1.0, 1.0).to(torch.float32)
    b = wl.Batch(logits, a, mu_logp, adv, None, None, None)
    dev = _run(b, dppo.BINARY_KL, 0, 0.01, dppo.KERNEL_AUTO)
    pin = lambda x: x.cpu().pin_memory()
    out = dppo.dppo_loss_fwd_bwd_host(pin(logits), pin(a), pin(mu_logp), pin(adv), None, dppo.BINARY_KL, 0, 0.01,
                                      rows_per_chunk=64, want_dlogits=True, device=DEV)
    assert out["status"] == 0
    assert torch.equal(out["divergence"], dev["divergence"].cpu()) and torch.equal(out["mask"], dev["mask"].cpu())
    a_, b_ = out["dlogits"].float(), dev["dlogits"].cpu().float()
    assert torch.all((a_ - b_).abs() <= 2.0 ** -7 * b_.abs())
    assert abs(out["loss"] - float(dev["loss"].item())) <= 1e-4 * abs(out["loss"]) + 1e-12


# ------------------------------------------------------------------------------------- very confident tokens

def _confident_rows(T, V, dtype, seed, K):
    """Rows whose distribution is dominated by one token (one logit at +16 ... +26 where the others have a log-sum-exp of
    about 7, so that 1 - pi of that token is 1e-4 ... 5e-9: beyond that the float64 oracle itself, which takes the
    complement as 1 - pi, runs out of digits), as LLM rollouts produce for most positions.  Three quarters of the rows sample the dominant token,
    the rest a random one.  The rollout side is taken from float64 (log-softmax of the noisy logits), so that the stored
    fp32 log-probabilities are exact roundings of probabilities below one."""
    g = torch.Generator(device=DEV).manual_seed(seed)
    z, _, _, _, _ = wl.logits_rows(0, T, V, torch.float32, seed, DEV, sigma=3.0, zipf=1.1, sigma_mu=0.1, K=0)
    col = torch.randint(0, V, (T,), generator=g, device=DEV)
    boost = 16.0 + 10.0 * torch.rand(T, generator=g, device=DEV)
    ar = torch.arange(T, device=DEV)
    z[ar, col] = boost
    zq = z.to(dtype)
    mu_logits = zq.double() + 0.3 * torch.randn((T, V), generator=g, device=DEV, dtype=torch.float64)
    logp = torch.log_softmax(mu_logits, dim=1)
    a = torch.where(ar % 4 != 3, col, torch.randint(0, V, (T,), generator=g, device=DEV))
    mu_logp = logp[ar, a].to(torch.float32).contiguous()
    top = torch.topk(logp, K, dim=1)
    ids, ps = top.indices.to(torch.int32).contiguous(), torch.exp(top.values).to(torch.float32).contiguous()
    adv = torch.where(ar % 2 == 0, 1.0, -1.0).to(torch.float32)
    return wl.Batch(zq, a.to(torch.int32), mu_logp, adv, None, ids, ps), (ar % 4 != 3).cpu().numpy()


@pytest.mark.parametrize("kernel", sorted(KERNELS))
@pytest.mark.parametrize("V,dtype", [(20008, torch.bfloat16), (4096, torch.float32), (151936, torch.bfloat16)])
def test_kl_of_very_confident_tokens_keeps_its_relative_accuracy(kernel, V, dtype):
    """Binary-KL needs 1 - pi(a); for a token with pi(a) = 1 - 1e-6 that complement must come from the sum over the other
    entries (1 - exp(z_a - lse) would lose it in the rounding of lse).  The KL values here are 1e-9 ... 1e-7, far below
    the 1e-5 absolute tolerance, so they are also held to a relative one."""
    T, K = 96, 8
    b, dominant = _confident_rows(T, V, dtype, seed=V % 97, K=K)
    h = P.host_inputs(b)
    for variant, k in ((dppo.BINARY_KL, 0), (dppo.TOPK_KL, K), (dppo.BINARY_TV, 0), (dppo.TOPK_TV, K)):
        out, ora, _ = _full_check(b, variant, k, 0.05, KERNELS[kernel], dlogits_f32=(dtype == torch.float32))
        if variant == dppo.BINARY_TV or variant == dppo.TOPK_TV:
            continue
        D = out["divergence"].cpu().numpy().astype(np.float64)
        # Top-K: the rows that sample the dominant token (it is in the list); the "other" mass of a row whose list holds a
        # dominant token that is not the sampled one is below what an fp32-accurate normaliser resolves (a documented limit)
        rows = np.nonzero(dominant)[0] if variant == dppo.TOPK_KL else np.arange(T)
        small = rows[ora["D"][rows] < 1e-6]
        assert len(small) > T // 2
        # (the float64 oracle, which forms 1 - pi by subtraction, is itself only good to a few 1e-16 here: rows whose two
        # policies nearly agree have a KL of that size, of either sign)
        err = np.abs(D[small] - ora["D"][small])
        assert np.all(err <= 1e-2 * np.abs(ora["D"][small]) + 1e-12), err.max()


# ------------------------------------------------------------------------------------- full size, the other runs of config 2

@pytest.mark.parametrize("variant,delta", [(dppo.BINARY_KL, 0.1), (dppo.BINARY_KL, 0.2), (dppo.BINARY_TV, 0.1)])
def test_full_size_binary_variants_sampled_rows(variant, delta):
    """Config 2's other three runs at T=16384, V=151936 (Binary-TV at delta=0.2 is the test above): sampled rows against
    the oracle, and the loss over a sixteenth of the rows."""
    T = 16384
    b = wl.qwen_vocab_rows(DEV, seed=1)
    out = _run(b, variant, 0, delta, dppo.KERNEL_AUTO)
    assert int(out["status"].item()) == 0
    rows = np.sort(np.random.default_rng(11 + variant).choice(T, 32, replace=False))
    h = P.host_inputs(b, rows)
    ora = P.run_oracle(h, variant, 0, delta, 1.0 / T)
    P.check_scalars(out["divergence"].cpu().numpy()[rows], out["mask"].cpu().numpy()[rows], ora, h, delta)
    P.check_dlogits(out["dlogits"][torch.as_tensor(rows, device=DEV)], ora["dlogits"], out_is_bf16=True,
                    max_abs=_grad_scale(b, 1.0 / T, ora, rows))
    tok = (torch.rand(T, generator=torch.Generator().manual_seed(6)) < 1.0 / 16).to(torch.uint8)
    idx = np.nonzero(tok.numpy())[0]
    bm = wl.Batch(b.logits, b.sampled_ids, b.mu_logp, b.advantages, tok.to(DEV))
    outm = _run(bm, variant, 0, delta, dppo.KERNEL_AUTO)
    hb = P.host_inputs(bm, idx)
    hb["token_mask"] = None
    ob = P.run_oracle(hb, variant, 0, delta, 1.0 / len(idx), want_grad=False)
    P.check_scalars(outm["divergence"].cpu().numpy()[idx], outm["mask"].cpu().numpy()[idx], ob, hb, delta)
    P.check_loss(float(outm["loss"].item()), ob["loss"], True, ob["row_loss"])


# ------------------------------------------------------------------------------------- config 4, the whole batch

def test_full_size_ragged_topk_kl_k64_whole_batch():
    """Config 4 as a whole: the 64 ragged responses (lengths uniform in [128, 8192], about 266 k valid rows, V=151936, K=64,
    rollout noise 0.3, TopK-KL, delta=0.05, the paper's KL threshold) streamed as 64 padded blocks of 8192 rows, each one
    call with the global token-mean scale 1 / (sum of lengths), the padding poisoned.  Per response: D, M and the gradient
    of sampled valid rows against the oracle, zeros in the padding.  For a stated subset of responses (the three shortest
    and one of medium length): the response's loss against the oracle over all its rows.  The batch loss is the fp64 sum
    of the 64 calls' losses; its subset part is compared with the oracle's."""
    lengths = wl.ragged_lengths()
    n_valid = int(sum(lengths))
    scale = 1.0 / n_valid
    order = np.argsort(lengths)
    subset = sorted(int(i) for i in list(order[:3]) + [int(order[len(order) // 2])])
    assert sum(lengths[i] for i in subset) <= 12000           # what the oracle does in well under a minute (forward only)
    rng = np.random.default_rng(17)
    dl = torch.empty((8192, wl.QWEN3_VOCAB), dtype=torch.bfloat16, device=DEV)
    ws = torch.empty(dppo.dppo_workspace_bytes(8192), dtype=torch.uint8, device=DEV)
    total_gpu, sub_gpu, sub_ora, blocked, rows_checked = 0.0, 0.0, 0.0, 0, 0
    for i in range(len(lengths)):
        L = int(lengths[i])
        b = wl.ragged_response(DEV, i, lengths)
        b.logits[L:] = float("nan")
        b.sampled_ids[L:] = -3
        b.mu_topk_ids[L:] = 1 << 28
        out = dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, b.token_mask, dppo.TOPK_KL, 64, 0.05,
                                     b.mu_topk_ids, b.mu_topk_p, loss_scale=scale, dlogits=dl, workspace=ws, want_stats=True)
        torch.cuda.synchronize()
        assert int(out["status"].item()) == 0 and out["stats"][0].item() == L
        loss_i = float(out["loss"].item())
        total_gpu += loss_i
        rows = np.sort(rng.choice(L, 8, replace=False))
        h = P.host_inputs(b, rows)
        h["token_mask"] = None
        ora = P.run_oracle(h, O.TOPK_KL, 64, 0.05, scale)
        P.check_scalars(out["divergence"].cpu().numpy()[rows], out["mask"].cpu().numpy()[rows], ora, h, 0.05)
        if np.abs(ora["dlogits"]).max() > 0:
            P.check_dlogits(dl[torch.as_tensor(rows, device=DEV)], ora["dlogits"], out_is_bf16=True)
        rows_checked += len(rows)
        pad = torch.arange(L, min(8192, L + 64), device=DEV)
        assert not dl[pad].any() and not out["mask"][L:].any() and not out["divergence"][L:].any()
        if i in subset:
            ora_loss, row_losses = 0.0, []
            Dg, Mg = out["divergence"].cpu().numpy(), out["mask"].cpu().numpy()
            for c0 in range(0, L, 512):                      # bounded host memory: 512 float64 rows at a time
                rr = np.arange(c0, min(L, c0 + 512))
                hs = P.host_inputs(b, rr)
                hs["token_mask"] = None
                os_ = P.run_oracle(hs, O.TOPK_KL, 64, 0.05, scale, want_grad=False)
                P.check_scalars(Dg[rr], Mg[rr], os_, hs, 0.05)
                ora_loss += os_["loss"]
                row_losses.append(os_["row_loss"])
                blocked += int((os_["M"] == 0).sum())
            # the scale is global, so a response's loss is small against the batch's; relative to its own size it must
            # still meet the bf16 tolerance
            P.check_loss(loss_i, ora_loss, True, np.concatenate(row_losses))
            sub_gpu += loss_i
            sub_ora += ora_loss
        del b, out
    assert rows_checked == 8 * len(lengths) and blocked > 0
    assert abs(sub_gpu - sub_ora) <= 1e-3 * abs(sub_ora)
    assert np.isfinite(total_gpu)


def test_host_buffer_entry_with_more_chunks_than_loss_slots():
    """One row per chunk and more chunks than the entry point keeps chunk losses on the device for (4096): the losses are
    collected in between and the total still matches the device entry point; one status word serves all chunks."""
    T, V = 4300, 520
    logits, a, mu_logp, _, _ = wl.logits_rows(0, T, V, torch.float32, 41, DEV, sigma=2.0, zipf=1.1, sigma_mu=0.3, K=0)
    adv = torch.where(torch.arange(T, device=DEV) % 3 == 0, -0.7, 1.0).to(torch.float32)
    tok = (torch.arange(T, device=DEV) % 11 != 5).to(torch.uint8)
    a = a.clone()
    a[4200] = V + 9                                   # a bad id in a late chunk: its status bit must reach the caller
    b = wl.Batch(logits, a, mu_logp, adv, tok, None, None)
    dev = _run(b, dppo.BINARY_KL, 0, 0.01, dppo.KERNEL_AUTO)
    pin = lambda x: x.cpu().pin_memory()
    out = dppo.dppo_loss_fwd_bwd_host(pin(logits), pin(a), pin(mu_logp), pin(adv), pin(tok), dppo.BINARY_KL, 0, 0.01,
                                      rows_per_chunk=1, want_dlogits=True, device=DEV)
    assert out["status"] == dppo.binding.STATUS_BAD_SAMPLED_ID == int(dev["status"].item())
    assert torch.equal(out["mask"], dev["mask"].cpu())
    assert torch.allclose(out["divergence"], dev["divergence"].cpu(), atol=1e-7, rtol=0)
    assert abs(out["loss"] - float(dev["loss"].item())) <= 1e-5 * abs(out["loss"]) + 1e-12
    a_, b_ = out["dlogits"], dev["dlogits"].cpu()
    assert torch.all((a_ - b_).abs() <= 1e-5 * b_.abs() + 1e-12)
