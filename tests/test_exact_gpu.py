"""Exact full-vocabulary TV / KL / entropy kernel against the float64 oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import paper_2602_04879_b200 as dppo
from oracle import dppo_oracle as O

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _pair(T, V, dtype, seed, noise):
    g = torch.Generator(device=DEV).manual_seed(seed)
    z = (3.0 * torch.randn((T, V), generator=g, device=DEV)).to(dtype)
    zm = (z.float() + noise * torch.randn((T, V), generator=g, device=DEV)).to(dtype)
    return z, zm


def _check(z, zm, tok=None, rows=None):
    out = dppo.dppo_exact_divergence(z, zm, tok)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    # without a TV output (tv = NULL) the second sweep is left out; KL and entropy are the same bits
    one = dppo.dppo_exact_divergence(z, zm, tok, want_tv=False)
    torch.cuda.synchronize()
    assert int(one["status"].item()) == 0 and one["tv"] is None
    assert torch.equal(one["kl"], out["kl"]) and torch.equal(one["entropy"], out["entropy"])
    T = z.shape[0]
    rows = range(T) if rows is None else rows
    zh, zmh = z.float().cpu().numpy().astype(np.float64), zm.float().cpu().numpy().astype(np.float64)
    tv, kl, ent = out["tv"].cpu().numpy(), out["kl"].cpu().numpy(), out["entropy"].cpu().numpy()
    for t in rows:
        if tok is not None and tok[t].item() == 0:
            assert tv[t] == 0 and kl[t] == 0 and ent[t] == 0
            continue
        o_tv, o_kl, o_ent = O.exact_divergence_row(zh[t], zmh[t])
        assert abs(tv[t] - o_tv) <= 1e-5 and abs(kl[t] - o_kl) <= 1e-5 and abs(ent[t] - o_ent) <= 2e-5 * max(1.0, o_ent), t
    return out


@pytest.mark.parametrize("T,V,dtype", [(37, 4096, torch.float32), (50, 1001, torch.bfloat16), (64, 151936, torch.bfloat16), (5, 8, torch.float32)])
def test_exact_divergence_matches_oracle(T, V, dtype):
    z, zm = _pair(T, V, dtype, seed=T + V, noise=0.5)
    tok = (torch.arange(T, device=DEV) % 5 != 2).to(torch.uint8)
    out = _check(z, zm, tok)
    # App. B: the Binary approximation never exceeds the exact divergence
    a = torch.randint(0, V, (T,), device=DEV, dtype=torch.int32)
    mu_logp = torch.log_softmax(zm.float(), 1).gather(1, a.long()[:, None])[:, 0].contiguous()
    adv = torch.ones(T, device=DEV)
    b_tv = dppo.dppo_loss_fwd_bwd(z, a, mu_logp, adv, tok, dppo.BINARY_TV, 0, 1.0)["divergence"]
    b_kl = dppo.dppo_loss_fwd_bwd(z, a, mu_logp, adv, tok, dppo.BINARY_KL, 0, 1.0)["divergence"]
    assert torch.all(b_tv <= out["tv"] + 1e-5) and torch.all(b_kl <= out["kl"] + 1e-5)


def test_exact_divergence_edge_cases():
    z, zm = _pair(8, 512, torch.float32, seed=3, noise=0.2)
    # identical policies: zero divergence, entropy of uniform logits = log V
    out = dppo.dppo_exact_divergence(z, z.clone())
    assert out["tv"].abs().max().item() <= 1e-6 and out["kl"].abs().max().item() <= 1e-6
    u = torch.zeros((3, 512), device=DEV)
    out = dppo.dppo_exact_divergence(u, u.clone())
    assert torch.allclose(out["entropy"], torch.full((3,), float(np.log(512)), device=DEV), atol=1e-5)
    # -inf entries are probability zero; a nan row only raises the status bit
    z2, zm2 = z.clone(), zm.clone()
    z2[:, 5::7] = float("-inf")
    zm2[:, 5::7] = float("-inf")
    _check(z2, zm2)
    z2[3, 0] = float("nan")
    out = dppo.dppo_exact_divergence(z2, zm2)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == dppo.binding.STATUS_NONFINITE_ROW and out["tv"][3].item() == 0
    # strided views
    wide = torch.zeros((8, 600), device=DEV)
    wide[:, :512] = z
    _check(wide[:, :512], zm)


@pytest.mark.parametrize("kernel", ["ring", "generic"])
@pytest.mark.parametrize("which,delta", [("tv", 0.1), ("kl", 0.03)])
def test_exact_divergence_as_the_trust_region(which, delta, kernel):
    """Variant GIVEN_D fed with the monitor's exact TV / KL: Eq. dppo_obj with the quantity the Sec. 4.4 forms
    approximate.  Against the oracle given the oracle's own exact values; the blocked set contains the Binary form's."""
    import parity_util as P
    from paper_2602_04879_b200 import workloads as wl
    T, V = 300, 4104
    z, zm = _pair(T, V, torch.bfloat16, seed=5, noise=0.6)
    g = torch.Generator(device=DEV).manual_seed(9)
    a = torch.multinomial(torch.softmax(zm.float(), 1), 1, generator=g)[:, 0].to(torch.int32)
    mu_logp = torch.log_softmax(zm.float(), 1).gather(1, a.long()[:, None])[:, 0].contiguous()
    adv = torch.where(torch.arange(T, device=DEV) % 2 == 0, 1.0, -0.5).to(torch.float32)
    tok = (torch.arange(T, device=DEV) % 6 != 4).to(torch.uint8)
    ex = dppo.dppo_exact_divergence(z, zm, tok, want_tv=(which == "tv"))
    code = dppo.KERNEL_RING if kernel == "ring" else dppo.KERNEL_GENERIC
    out = dppo.dppo_loss_fwd_bwd(z, a, mu_logp, adv, tok, dppo.GIVEN_D, 0, delta, kernel=code, given_divergence=ex[which],
                                 dlogits_f32=True)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    b = wl.Batch(z, a, mu_logp, adv, tok, None, None)
    h = P.host_inputs(b)
    zh, zmh = h["logits"], zm.float().cpu().numpy().astype(np.float64)
    full = np.array([O.exact_divergence_row(zh[t], zmh[t])[0 if which == "tv" else 1] if h["token_mask"][t] else 0.0 for t in range(T)])
    ora = P.run_oracle(h, O.GIVEN_D, 0, delta, None, given_D=full)
    P.check_scalars(out["divergence"].cpu().numpy(), out["mask"].cpu().numpy(), ora, h, delta)
    P.check_loss(float(out["loss"].item()), ora["loss"], True, ora["row_loss"])
    P.check_dlogits(out["dlogits"], ora["dlogits"], out_is_bf16=False)
    valid = h["token_mask"] != 0
    blocked = int(((ora["M"] == 0) & valid).sum())
    assert 0 < blocked < int(valid.sum())
    binary = dppo.dppo_loss_fwd_bwd(z, a, mu_logp, adv, tok, dppo.BINARY_TV if which == "tv" else dppo.BINARY_KL, 0, delta, kernel=code)
    assert torch.all(out["mask"] <= binary["mask"])          # App. B: D_bin <= D_full, so the exact region blocks a superset



def test_exact_kl_only_full_vocabulary_many_rows():
    """The one-sweep mode (KL and entropy, no TV) on more rows than CTAs at V=151936: several rows per CTA back to back,
    where the warps' partials of consecutive rows alternate between two buffers."""
    T, V = 700, 151936
    z, zm = _pair(T, V, torch.bfloat16, seed=77, noise=0.3)
    tok = (torch.arange(T, device=DEV) % 9 != 4).to(torch.uint8)
    one = dppo.dppo_exact_divergence(z, zm, tok, want_tv=False)
    two = dppo.dppo_exact_divergence(z, zm, tok)
    torch.cuda.synchronize()
    assert int(one["status"].item()) == 0 and torch.equal(one["kl"], two["kl"]) and torch.equal(one["entropy"], two["entropy"])
    rows = [0, 1, 147, 148, 149, 295, 296, 443, 592, 699]
    zh, zmh = z[rows].float().cpu().numpy().astype(np.float64), zm[rows].float().cpu().numpy().astype(np.float64)
    for i, t in enumerate(rows):
        if tok[t].item() == 0:
            assert one["kl"][t].item() == 0 and one["entropy"][t].item() == 0
            continue
        o_tv, o_kl, o_ent = O.exact_divergence_row(zh[i], zmh[i])
        assert abs(one["kl"][t].item() - o_kl) <= 1e-5 and abs(one["entropy"][t].item() - o_ent) <= 2e-5 * max(1.0, o_ent)
        assert abs(two["tv"][t].item() - o_tv) <= 1e-5
