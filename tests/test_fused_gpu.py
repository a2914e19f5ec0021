"""Fused LM-head variant on the GPU: the tensor-core GEMM building block, then the whole variant against the oracle."""
import numpy as np
import pytest
import torch

import paper_2602_04879_b200 as dppo
from paper_2602_04879_b200 import workloads as wl
from oracle import dppo_oracle as O

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
DW_ROUNDING = 2.0 ** -7            # entrywise bound on dW relative to |H|^T |dlogits|: two bf16 roundings, see _check_fused


@pytest.fixture(params=[2, 1], ids=["cta_pair", "single_cta"])
def cta_group(request):
    """Both modes of the tensor-core GEMM (opts.gemm_cta_group): pairs of SMs (the default) and single SMs."""
    return request.param


@pytest.fixture(params=[0, 128], ids=["all_rows_at_once", "row_blocks_of_128"])
def rows_per_block(request):
    """opts.fused_rows_per_block: the whole batch at once, or finished in blocks of 128 rows (bounded workspace)."""
    return request.param


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 256, 256), (300, 520, 200), (256, 1024, 1024), (1000, 264, 4104)])
def test_gemm_tn_bf16_matches_fp64_product(M, N, K, cta_group):
    g = torch.Generator(device=DEV).manual_seed(M * 7 + N * 3 + K)
    A = torch.randn((M, K), generator=g, device=DEV).to(torch.bfloat16)
    B = torch.randn((N, K), generator=g, device=DEV).to(torch.bfloat16)
    C, status = dppo.dppo_gemm_tn_bf16(A, B, cta_group=cta_group)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = A.double().cpu().numpy() @ B.double().cpu().numpy().T          # exact bf16 products, float64 accumulation
    err = np.abs(C.cpu().numpy() - ref).max()
    assert err <= 2e-5 * np.abs(ref).max() + 1e-4, err
    # strided operands (views into wider buffers) and a strided output
    Aw = torch.zeros((M, K + 24), dtype=torch.bfloat16, device=DEV)
    Aw[:, :K] = A
    Cw = torch.full((M, N + 5), 7.0, dtype=torch.float32, device=DEV)
    dppo.dppo_gemm_tn_bf16(Aw[:, :K], B, C=Cw[:, :N], cta_group=cta_group)
    torch.cuda.synchronize()
    assert torch.equal(Cw[:, :N], C) and torch.all(Cw[:, N:] == 7.0)


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 256, 256), (300, 520, 200), (256, 1024, 1024), (264, 4104, 1000)])
def test_gemm_nn_bf16_matches_fp64_product(M, N, K, cta_group):
    """B given as [K, N]: the MN-major operand path of the tensor-core GEMM."""
    g = torch.Generator(device=DEV).manual_seed(M * 5 + N * 11 + K)
    A = torch.randn((M, K), generator=g, device=DEV).to(torch.bfloat16)
    B = torch.randn((K, N), generator=g, device=DEV).to(torch.bfloat16)
    C, status = dppo.dppo_gemm_nn_bf16(A, B, cta_group=cta_group)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = A.double().cpu().numpy() @ B.double().cpu().numpy()
    err = np.abs(C.cpu().numpy() - ref).max()
    assert err <= 2e-5 * np.abs(ref).max() + 1e-4, err


def _fused_case(T, d, V, seed, resp_len, K=0, sigma_w=None):
    sw = 0.02 * (2048 / d) ** 0.5 if sigma_w is None else sigma_w
    return wl.lm_head_workload(DEV, seed=seed, T=T, d=d, V=V, resp_len=resp_len, sigma_w=sw, K=K)


def _check_fused(b, variant, delta, tok=None, K=0, is_cap=0.0, cta_group=0, rows_per_block=0, two_pass=False):
    T_, d_ = b.hidden.shape
    ws = None
    if rows_per_block:      # exactly the bounded workspace, poisoned: a kernel that reached beyond it or relied on its contents would show
        ws = torch.full((dppo.dppo_fused_workspace_bytes(min(T_, rows_per_block), d_, b.lm_head.shape[1], K),), 0xFF, dtype=torch.uint8, device=DEV)
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, tok, variant, delta,
                                         want_stats=True, K=K, mu_topk_ids=b.mu_topk_ids, mu_topk_p=b.mu_topk_p, is_cap=is_cap,
                                         cta_group=cta_group, rows_per_block=rows_per_block, workspace=ws, two_pass=two_pass)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    H = b.hidden.float().cpu().numpy().astype(np.float64)
    W = b.lm_head.float().cpu().numpy().astype(np.float64)
    tokh = None if tok is None else tok.cpu().numpy()
    ora = O.dppo_fused_lmhead_fwd_bwd(H, W, b.sampled_ids.cpu().numpy(), b.mu_logp.cpu().numpy().astype(np.float64),
                                      b.advantages.cpu().numpy().astype(np.float64), tokh, variant, delta, None, K,
                                      None if b.mu_topk_ids is None else b.mu_topk_ids.cpu().numpy(),
                                      None if b.mu_topk_p is None else b.mu_topk_p.cpu().numpy().astype(np.float64),
                                      is_cap if is_cap > 0 else None)
    h = dict(token_mask=tokh)
    P.check_scalars(out["divergence"].cpu().numpy(), out["mask"].cpu().numpy(), ora, h, delta)
    P.check_loss(float(out["loss"].item()), ora["loss"], True, ora["row_loss"])
    # The exponentials behind dlogits are rounded to bf16 before the two gradient GEMMs (8 significant bits: relative error
    # <= 2^-8 each) and, for dW, so are the hidden rows once they carry their row factor (another 2^-8).  Entrywise bounds:
    # 2^-8 (|P| |W|^T) for dHidden and 2^-7 (|H|^T |P|) for dW; entries that one term dominates (the sampled token's
    # column) come close to them, the fp32 arithmetic in front of the roundings is covered by the additive term
    aP = np.abs(ora["dlogits"])
    bound_h = 2.0 ** -8 * (aP @ np.abs(W).T) + 1e-7 * np.abs(ora["dHidden"]).max()
    # (the two-pass mode rounds the finished gradient once and leaves the hidden rows as they are: half the bound)
    bound_w = (0.5 if two_pass else 1.0) * DW_ROUNDING * (np.abs(H).T @ aP) + 1e-7 * np.abs(ora["dW"]).max()
    eh = np.abs(out["dHidden"].cpu().numpy() - ora["dHidden"])
    ew = np.abs(out["dW"].cpu().numpy() - ora["dW"])
    assert np.all(eh <= bound_h), (eh / bound_h).max()
    assert np.all(ew <= bound_w), (ew / bound_w).max()
    # and in aggregate the error is far below the bound
    assert eh.max() <= 4e-3 * np.abs(ora["dHidden"]).max() and ew.max() <= 8e-3 * np.abs(ora["dW"]).max()
    valid = np.ones(T_, bool) if tokh is None else tokh != 0
    st = out["stats"].cpu().numpy()
    assert st[0] == valid.sum() and st[1] == int(((ora["M"] == 0) & valid).sum())
    assert abs(st[5] - ora["r"][valid].sum()) <= 1e-3 * max(1.0, st[5])
    return out, ora


@pytest.mark.parametrize("T,d,V", [(256, 128, 1024), (200, 72, 1000), (384, 256, 2304)])
def test_fused_matches_oracle_small(T, d, V, cta_group, rows_per_block):
    b = _fused_case(T, d, V, seed=41, resp_len=8)
    kw = dict(cta_group=cta_group, rows_per_block=rows_per_block)
    out, ora = _check_fused(b, dppo.BINARY_TV, 0.2, **kw)
    # mask stress near the median divergence, KL variant, ragged mask
    Dm = np.sort(ora["D"])
    delta = float(np.float32(0.5 * (Dm[len(Dm) // 2] + Dm[len(Dm) // 2 + 1])))
    tok = (torch.arange(T, device=DEV) % 7 != 3).to(torch.uint8)
    out2, ora2 = _check_fused(b, dppo.BINARY_TV, delta, tok, **kw)
    valid = tok.cpu().numpy() != 0
    assert 0 < int(((ora2["M"] == 0) & valid).sum()) < int(valid.sum())
    _check_fused(b, dppo.BINARY_KL, 1e-9, tok, **kw)


def test_fused_two_pass_mode_rounds_the_gradient_once(cta_group, rows_per_block):
    """opts.fused_two_pass: every row through the statistics GEMM and the gradient GEMM (each logits tile computed twice);
    dW then carries one bf16 rounding, and meets half the entrywise bound of the single-pass route."""
    T, d, V, K = 384, 256, 2304, 6
    b = _fused_case(T, d, V, seed=45, resp_len=8, K=K, sigma_w=0.3)
    tok = (torch.arange(T, device=DEV) % 7 != 3).to(torch.uint8)
    adv = b.advantages.clone()
    adv[(torch.arange(T, device=DEV) // 8) % 4 == 1] = 0.0
    b.advantages = adv
    kw = dict(cta_group=cta_group, rows_per_block=rows_per_block, two_pass=True)
    out, ora = _check_fused(b, dppo.BINARY_TV, 0.2, **kw)
    Dm = np.sort(ora["D"])
    delta = float(np.float32(0.5 * (Dm[T // 2] + Dm[T // 2 + 1])))
    out2, ora2 = _check_fused(b, dppo.BINARY_KL, delta * delta, tok, **kw)
    _check_fused(b, dppo.TOPK_TV, 0.01, tok, K=K, **kw)
    one = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, tok, dppo.BINARY_KL, delta * delta,
                                         cta_group=cta_group, rows_per_block=rows_per_block)
    torch.cuda.synchronize()
    assert torch.equal(one["mask"], out2["mask"]) and torch.allclose(one["divergence"], out2["divergence"], atol=2e-6, rtol=0)


@pytest.mark.parametrize("variant", [dppo.TOPK_TV, dppo.TOPK_KL])
def test_fused_topk_variants_match_oracle(variant, rows_per_block):
    """Top-K divergences in the fused path: peaked logits (larger LM-head scale) so that the top-K lists carry mass."""
    T, d, V, K = 256, 128, 2048, 20
    b = _fused_case(T, d, V, seed=43, resp_len=8, K=K, sigma_w=0.35)
    out, ora = _check_fused(b, variant, 1.0, K=K, rows_per_block=rows_per_block)
    Dm = np.sort(ora["D"])
    gaps = Dm[T // 2 - 6:T // 2 + 6]
    i = int(np.argmax(np.diff(gaps)))
    delta = float(np.float32(0.5 * (gaps[i] + gaps[i + 1])))
    tok = (torch.arange(T, device=DEV) % 5 != 1).to(torch.uint8)
    out2, ora2 = _check_fused(b, variant, delta, tok, K=K, is_cap=1.05, rows_per_block=rows_per_block)
    valid = tok.cpu().numpy() != 0
    assert 0 < int(((ora2["M"] == 0) & valid).sum()) < int(valid.sum())
    # App. B: Top-K refines Binary
    bin_out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, variant - 2, 1.0)
    assert torch.all(bin_out["divergence"] <= out["divergence"] + 1e-5)      # equality happens; 1e-5 is the tolerance of D
    # an out-of-range list entry raises the status bit and drops the row
    bad = b.mu_topk_ids.clone()
    bad[7, 3] = V + 5
    o3 = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, variant, 1.0,
                                        K=K, mu_topk_ids=bad, mu_topk_p=b.mu_topk_p)
    torch.cuda.synchronize()
    assert int(o3["status"].item()) == dppo.binding.STATUS_BAD_TOPK_ID and not o3["dHidden"][7].any()


def test_fused_backward_skips_rows_without_gradient(cta_group, rows_per_block):
    """Invalid rows drop out of every GEMM and rows with zero advantage out of the backward GEMMs (the kept rows are packed
    on the device); rows blocked by the mask stay in with a zero factor.  The outputs must not show any of this: zeros in
    dHidden for all those rows, the same dW."""
    T, d, V = 600, 128, 1536
    b = _fused_case(T, d, V, seed=47, resp_len=8)
    adv = b.advantages.clone()
    adv[(torch.arange(T, device=DEV) // 8) % 3 == 0] = 0.0           # every third response has zero advantage
    b.advantages = adv
    kw = dict(cta_group=cta_group, rows_per_block=rows_per_block)
    out0, ora0 = _check_fused(b, dppo.BINARY_TV, 0.2, **kw)
    Dm = np.sort(ora0["D"])
    delta = float(np.float32(0.5 * (Dm[T // 2] + Dm[T // 2 + 1])))
    tok = (torch.arange(T, device=DEV) % 11 != 4).to(torch.uint8)
    out, ora = _check_fused(b, dppo.BINARY_TV, delta, tok, **kw)
    zero = (ora["M"] == 0) | (tok.cpu().numpy() == 0) | (adv.cpu().numpy() == 0)
    kept = int((~zero).sum())
    assert 0 < kept < T and kept % 64 != 0
    assert not out["dHidden"][torch.from_numpy(zero).to(DEV)].any()
    assert out["dHidden"][torch.from_numpy(~zero).to(DEV)].abs().sum(dim=1).min().item() > 0
    # nothing left at all: zero advantages everywhere
    b.advantages = torch.zeros_like(adv)
    o2 = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, tok, dppo.BINARY_TV, delta, **kw)
    torch.cuda.synchronize()
    assert int(o2["status"].item()) == 0 and float(o2["loss"].item()) == 0.0
    assert not o2["dHidden"].any() and not o2["dW"].any()
    assert np.array_equal(o2["divergence"].cpu().numpy(), out["divergence"].cpu().numpy())
    # no valid row at all
    o3 = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, adv, torch.zeros_like(tok), dppo.BINARY_TV, delta, **kw)
    torch.cuda.synchronize()
    assert int(o3["status"].item()) == 0 and not o3["dHidden"].any() and not o3["dW"].any() and not o3["mask"].any()


def test_fused_rows_with_a_vanishing_sampled_token_take_the_two_pass_route(rows_per_block):
    """The single forward pass measures every logit against the sampled token's logit.  Rows whose sampled token has a
    probability below 2^-60 under the trainer policy (sum of exponentials out of the safe range, or beyond fp32
    altogether) are recomputed by the two-pass kernels; the results must match the oracle like any other row."""
    T, d, V = 300, 128, 1536
    b = _fused_case(T, d, V, seed=53, resp_len=4, sigma_w=0.35, K=8)      # logits ~ N(0, 4^2)
    rows = torch.tensor([3, 64, 65, 130, 255, 299], device=DEV)
    hid = b.hidden.clone()
    hid[rows] = hid[rows] * torch.tensor([4, 4, 8, 8, 8, 4], device=DEV, dtype=hid.dtype)[:, None]   # spreads of +-50 / +-100
    b.hidden = hid
    z = b.hidden.double() @ b.lm_head.double()                            # input construction only
    lsm = torch.log_softmax(z, dim=1)
    ids = b.sampled_ids.clone()
    mu = b.mu_logp.clone()
    ids[rows] = torch.argmin(z[rows], dim=1).to(ids.dtype)               # the least likely token of the row
    lp = lsm[rows, ids[rows].long()]
    assert float(lp.max()) < -60.0 and float(lp.min()) < -100.0           # below 2^-60, some beyond exp's fp32 range
    # a rollout probability of the same size, so that the ratio is of order one and the row has a real gradient
    mu[rows] = (lp + 0.3 * torch.tensor([1, -1, 1, -1, 1, -1], device=DEV)).float()
    b.sampled_ids, b.mu_logp = ids, mu
    adv = b.advantages.clone()
    adv[299] = 0.0                                                        # one of them without gradient
    adv[296:299] = 0.0
    b.advantages = adv
    kw = dict(rows_per_block=rows_per_block)
    for variant, delta in ((dppo.BINARY_TV, 0.2), (dppo.BINARY_KL, 0.05)):
        out, ora = _check_fused(b, variant, delta, **kw)
        g_rows = np.abs(ora["dlogits"][rows.cpu().numpy()[:-1]]).max(axis=1)
        assert g_rows.min() > 1e-2 * np.abs(ora["dlogits"]).max()        # the recomputed rows matter in dW and dHidden
    tok = (torch.arange(T, device=DEV) % 9 != 2).to(torch.uint8)         # row 65 invalid, 299 invalid
    _check_fused(b, dppo.BINARY_TV, 0.2, tok, **kw)
    # the two-pass route with a Top-K divergence (TV: on these extremely peaked rows the "other" mass of pi is ~1e-12,
    # below what an fp32-accurate normaliser resolves, so the KL form's log of it is not a fair comparison)
    _check_fused(b, dppo.TOPK_TV, 0.05, tok, K=8, **kw)
    # a non-finite hidden row is reported, dropped, and does not leak into dW
    hid = b.hidden.clone()
    hid[10, 5] = float("inf")
    o = dppo.dppo_fused_lmhead_fwd_bwd(hid, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0.2, **kw)
    torch.cuda.synchronize()
    assert int(o["status"].item()) == dppo.binding.STATUS_NONFINITE_ROW
    assert not o["dHidden"][10].any() and int(o["mask"][10].item()) == 0
    assert torch.isfinite(o["dW"]).all() and torch.isfinite(o["dHidden"]).all()
    # a row with an out-of-range sampled id next to logits beyond exp's fp32 range: the row is reported and dropped before
    # it gets a row of exponentials (taken against reference 0 they would overflow and poison dW and dHidden through 0 * inf)
    ids = b.sampled_ids.clone()
    ids[64] = V + 3
    ids[130] = -1
    o = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0.2, **kw)
    torch.cuda.synchronize()
    assert float((b.hidden[130].double() @ b.lm_head.double()).max()) > 89.0          # e^89 > FLT_MAX
    assert int(o["status"].item()) == dppo.binding.STATUS_BAD_SAMPLED_ID
    assert torch.isfinite(o["dW"]).all() and torch.isfinite(o["dHidden"]).all()
    assert not o["dHidden"][64].any() and not o["dHidden"][130].any() and int(o["mask"][64].item()) == 0
    keep = torch.ones(T, dtype=torch.uint8, device=DEV)
    keep[64] = 0
    keep[130] = 0
    ref = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, keep, dppo.BINARY_TV, 0.2,
                                         loss_scale=1.0 / T, **kw)
    torch.cuda.synchronize()
    # same rows in the same packed order; the scale is 1/T in double in one call and the fp32 argument in the other
    assert torch.allclose(o["dW"], ref["dW"], rtol=1e-2, atol=1e-6 * float(ref["dW"].abs().max().item()))
    assert torch.allclose(o["dHidden"], ref["dHidden"], rtol=1e-5, atol=0)


@pytest.mark.parametrize("T,d,V", [(1, 8, 8), (7, 16, 264), (65, 8, 520)])
def test_fused_tiny_shapes(T, d, V):
    """Fewer rows than one K block of the dW GEMM, one row, one tile: the padded parts of the staged operands must not leak."""
    b = _fused_case(T, d, V, seed=59, resp_len=1, sigma_w=0.5)
    poison = torch.full((dppo.dppo_fused_workspace_bytes(T, d, V),), 0xFF, dtype=torch.uint8, device=DEV)   # NaN patterns
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0.2,
                                         workspace=poison)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    assert torch.isfinite(out["dW"]).all() and torch.isfinite(out["dHidden"]).all()
    _check_fused(b, dppo.BINARY_TV, 0.2)
    _check_fused(b, dppo.BINARY_KL, 0.0)
    # row blocks that leave a last block of one row (T = 65), blocks of one row, and the two-pass mode on the same shapes
    _check_fused(b, dppo.BINARY_TV, 0.2, rows_per_block=64)
    _check_fused(b, dppo.BINARY_KL, 0.0, rows_per_block=1 if T <= 7 else 16)
    _check_fused(b, dppo.BINARY_TV, 0.2, two_pass=True, rows_per_block=64)


@pytest.mark.parametrize("T,d,V,K", [(256, 128, 1024, 0), (300, 72, 1000, 6), (520, 136, 2056, 0)])
def test_fused_with_the_lm_head_stored_vocabulary_major(T, d, V, K, cta_group, rows_per_block):
    """W given as [V, d] (how a linear layer stores its weight) and dW returned in that layout: same results as with [d, V]."""
    b = _fused_case(T, d, V, seed=71, resp_len=4, K=K, sigma_w=0.3 if K else None)
    variant = dppo.TOPK_TV if K else dppo.BINARY_TV
    tok = (torch.arange(T, device=DEV) % 7 != 2).to(torch.uint8)
    kw = dict(K=K, mu_topk_ids=b.mu_topk_ids, mu_topk_p=b.mu_topk_p, cta_group=cta_group, rows_per_block=rows_per_block)
    ref, ora = _check_fused(b, variant, 0.01, tok, K=K, cta_group=cta_group, rows_per_block=rows_per_block)
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head.t().contiguous(), b.sampled_ids, b.mu_logp, b.advantages, tok, variant, 0.01,
                                         w_is_vd=True, **kw)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0 and out["dW"].shape == (V, d)
    assert torch.equal(out["mask"], ref["mask"])
    assert torch.allclose(out["divergence"], ref["divergence"], atol=2e-6, rtol=0)
    H = b.hidden.float().cpu().numpy().astype(np.float64)
    W = b.lm_head.float().cpu().numpy().astype(np.float64)
    aP = np.abs(ora["dlogits"])
    eh = np.abs(out["dHidden"].cpu().numpy() - ora["dHidden"])
    ew = np.abs(out["dW"].cpu().numpy().T - ora["dW"])
    assert np.all(eh <= 2.0 ** -8 * (aP @ np.abs(W).T) + 1e-7 * np.abs(ora["dHidden"]).max())
    assert np.all(ew <= DW_ROUNDING * (np.abs(H).T @ aP) + 1e-7 * np.abs(ora["dW"]).max())
    P.check_loss(float(out["loss"].item()), ora["loss"], True, ora["row_loss"])


def test_fused_with_a_given_divergence():
    """Variant GIVEN_D through the LM-head path: the caller's per-token divergence decides the mask."""
    T, d, V = 260, 128, 1032
    b = _fused_case(T, d, V, seed=67, resp_len=4, sigma_w=0.3)
    g = torch.Generator(device=DEV).manual_seed(3)
    Dg = torch.rand(T, generator=g, device=DEV) * 0.2
    tok = (torch.arange(T, device=DEV) % 5 != 3).to(torch.uint8)
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, tok, dppo.GIVEN_D, 0.1,
                                         given_divergence=Dg)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    H = b.hidden.float().cpu().numpy().astype(np.float64)
    W = b.lm_head.float().cpu().numpy().astype(np.float64)
    tokh = tok.cpu().numpy()
    ora = O.dppo_fused_lmhead_fwd_bwd(H, W, b.sampled_ids.cpu().numpy(), b.mu_logp.cpu().numpy().astype(np.float64),
                                      b.advantages.cpu().numpy().astype(np.float64), tokh, O.GIVEN_D, 0.1,
                                      given_D=Dg.cpu().numpy().astype(np.float64))
    P.check_scalars(out["divergence"].cpu().numpy(), out["mask"].cpu().numpy(), ora, dict(token_mask=tokh), 0.1)
    P.check_loss(float(out["loss"].item()), ora["loss"], True, ora["row_loss"])
    assert 0 < int(((ora["M"] == 0) & (tokh != 0)).sum()) < int((tokh != 0).sum())
    ew = np.abs(out["dW"].cpu().numpy() - ora["dW"])
    assert np.all(ew <= DW_ROUNDING * (np.abs(H).T @ np.abs(ora["dlogits"])) + 1e-7 * np.abs(ora["dW"]).max())


def test_fused_is_deterministic(cta_group, rows_per_block):
    """Same inputs, same bits: the only atomics of the path add two partial sums into zeros, which commutes; the row
    blocks add their parts of dW and of the loss in stream order."""
    b = _fused_case(520, 136, 2056, seed=61, resp_len=8, K=4)
    tok = (torch.arange(520, device=DEV) % 6 != 1).to(torch.uint8)
    runs = []
    for _ in range(3):
        o = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, tok, dppo.TOPK_KL, 0.001,
                                           K=4, mu_topk_ids=b.mu_topk_ids, mu_topk_p=b.mu_topk_p, cta_group=cta_group,
                                           rows_per_block=rows_per_block)
        torch.cuda.synchronize()
        runs.append(o)
    for o in runs[1:]:
        for key in ("loss", "divergence", "mask", "dHidden", "dW"):
            assert torch.equal(o[key], runs[0][key]), key


def test_fused_rejects_misuse():
    b = _fused_case(128, 64, 512, seed=42, resp_len=8)
    with pytest.raises(dppo.DppoError) as e:
        dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.TOPK_TV, 0.2, K=4)
    assert e.value.code == -5
    with pytest.raises(dppo.DppoError) as e:
        dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, 9, 0.2)
    assert e.value.code == -4
    with pytest.raises(dppo.DppoError) as e:
        dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0.2,
                                       workspace=torch.empty(1024, dtype=torch.uint8, device=DEV))
    assert e.value.code == -8


def test_fused_full_size_masked_subset_and_properties():
    """The benchmark's fused configuration (T=8192, d=2048, V=151936).  (i) With a token mask that keeps 192 rows the
    oracle can do everything: loss, mask, divergence, dHidden of the valid rows and the whole dW.  (ii) With all rows
    valid: sampled rows against the oracle, and properties that hold at any size."""
    T, d, V = 8192, 2048, 151936
    b = wl.lm_head_workload(DEV, seed=5)
    assert b.hidden.shape == (T, d) and b.lm_head.shape == (d, V)
    ws = torch.empty(dppo.dppo_fused_workspace_bytes(T, d, V), dtype=torch.uint8, device=DEV)
    W64 = b.lm_head.float().cpu().numpy().astype(np.float64)
    # ---- (i) masked subset
    g = torch.Generator().manual_seed(9)
    keep = torch.sort(torch.randperm(T, generator=g)[:192]).values
    tok = torch.zeros(T, dtype=torch.uint8)
    tok[keep] = 1
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, tok.to(DEV),
                                         dppo.BINARY_TV, 0.0, workspace=ws, want_stats=True)   # delta = 0: blocked iff moving away
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0 and out["stats"][0].item() == 192
    idx = keep.numpy()
    Hk = b.hidden[keep.to(DEV)].float().cpu().numpy().astype(np.float64)
    ora = O.dppo_fused_lmhead_fwd_bwd(Hk, W64, b.sampled_ids.cpu().numpy()[idx], b.mu_logp.cpu().numpy().astype(np.float64)[idx],
                                      b.advantages.cpu().numpy().astype(np.float64)[idx], None, O.BINARY_TV, 0.0, 1.0 / 192)
    # the logits of this workload are nearly uniform (D ~ 1e-6), so every row is inside the 1e-6 exemption band of the
    # divergence test; the masks are compared directly instead (the decision is the sign of log pi(a) - log mu(a))
    P.check_scalars(out["divergence"].cpu().numpy()[idx], out["mask"].cpu().numpy()[idx], ora, dict(token_mask=None), 0.0)
    assert np.array_equal(out["mask"].cpu().numpy()[idx], ora["M"])
    assert 0 < int((ora["M"] == 0).sum()) < 192
    P.check_loss(float(out["loss"].item()), ora["loss"], True, ora["row_loss"])
    aP = np.abs(ora["dlogits"])
    eh = np.abs(out["dHidden"][keep.to(DEV)].cpu().numpy() - ora["dHidden"])
    assert np.all(eh <= 2.0 ** -8 * (aP @ np.abs(W64).T) + 1e-7 * np.abs(ora["dHidden"]).max())
    ew = np.abs(out["dW"].cpu().numpy() - ora["dW"])
    assert np.all(ew <= DW_ROUNDING * (np.abs(Hk).T @ aP) + 1e-7 * np.abs(ora["dW"]).max())
    assert eh.max() <= 4e-3 * np.abs(ora["dHidden"]).max() and ew.max() <= 8e-3 * np.abs(ora["dW"]).max()
    inv = torch.nonzero(tok == 0)[:, 0][:256].to(DEV)
    assert not out["dHidden"][inv].any() and not out["divergence"][inv].any()
    del ora, aP, eh, ew
    # ---- (ii) all rows valid (the benchmark's launch configuration): the forward of every row in float64, dW element-wise on
    # a sample of columns (each a dot product over all T = 8192 rows: the dW GEMM's whole K loop), dHidden on sampled rows
    del out
    _check_all_valid_full_size(b, W64, ws, rows_per_block=0)


_ORACLE_CACHE = {}       # the float64 forward of all 8192 rows takes the host a minute or two: both full-size tests share it


def _check_all_valid_full_size(b, W64, ws, rows_per_block):
    T, d = b.hidden.shape
    V = b.lm_head.shape[1]
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None,
                                         dppo.BINARY_TV, 0.2, workspace=ws, want_stats=True, rows_per_block=rows_per_block)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0 and out["stats"][0].item() == T
    g = torch.Generator().manual_seed(12)
    ids = b.sampled_ids.cpu().numpy()
    cols = np.unique(np.concatenate([torch.randint(0, V, (56,), generator=g).numpy(), ids[::1024]]))      # sampled-token columns too
    rows = np.sort(torch.randperm(T, generator=g)[:24].numpy())
    H64 = b.hidden.float().cpu().numpy().astype(np.float64)
    key = (T, d, V, int(ids[:64].sum()), float(b.hidden[:8].float().sum().item()))
    if key not in _ORACLE_CACHE:
        _ORACLE_CACHE[key] = O.dppo_fused_lmhead_sampled(H64, W64, ids, b.mu_logp.cpu().numpy().astype(np.float64),
                                                         b.advantages.cpu().numpy().astype(np.float64), None, O.BINARY_TV, 0.2,
                                                         None, cols, rows)
    ora = _ORACLE_CACHE[key]
    P.check_scalars(out["divergence"].cpu().numpy(), out["mask"].cpu().numpy(), ora, dict(token_mask=None), 0.2)
    P.check_loss(float(out["loss"].item()), ora["loss"], True, ora["row_loss"])
    assert len(cols) >= 64
    dWc = out["dW"][:, torch.as_tensor(cols, device=DEV)].cpu().numpy().astype(np.float64)
    ew = np.abs(dWc - ora["dW_cols"])
    bound_w = DW_ROUNDING * (np.abs(H64).T @ np.abs(ora["dlogits_cols"])) + 1e-7 * np.abs(ora["dW_cols"]).max()
    assert np.all(ew <= bound_w), (ew / bound_w).max()
    assert ew.max() <= 8e-3 * np.abs(ora["dW_cols"]).max()
    eh = np.abs(out["dHidden"][torch.as_tensor(rows, device=DEV)].cpu().numpy() - ora["dHidden_rows"])
    assert np.all(eh <= 2.0 ** -8 * (np.abs(ora["dlogits_rows"]) @ np.abs(W64).T) + 1e-7 * np.abs(ora["dHidden_rows"]).max())
    assert eh.max() <= 4e-3 * np.abs(ora["dHidden_rows"]).max()
    # every dlogits row sums to zero, hence every row of dW does (up to the bf16 rounding of dlogits)
    dW = out["dW"]
    scale_w = float(dW.abs().sum(dim=1).max().item())
    assert float(dW.sum(dim=1).abs().max().item()) <= 5e-3 * scale_w
    assert torch.isfinite(out["dHidden"]).all() and torch.isfinite(dW).all()
    return out


def test_fused_full_size_in_row_blocks_with_a_bounded_workspace():
    """The fused configuration finished in blocks of 2048 rows: the workspace is that of 2048 rows (the 2.49 GB of staged
    exponentials of the whole batch are never there), the results meet the same bounds as at once, twice the same bits;
    and a batch four times as long (T = 32768) runs in the same workspace."""
    T, d, V, R = 8192, 2048, 151936, 2048
    b = wl.lm_head_workload(DEV, seed=5)
    need = dppo.dppo_fused_workspace_bytes(R, d, V)
    assert need < 0.9e9 and need == dppo.dppo_fused_workspace_bytes(min(T, R), d, V) and dppo.dppo_fused_workspace_bytes(T, d, V) > 2.4e9
    ws = torch.full((need,), 0xFF, dtype=torch.uint8, device=DEV)
    W64 = b.lm_head.float().cpu().numpy().astype(np.float64)
    out = _check_all_valid_full_size(b, W64, ws, rows_per_block=R)
    del W64
    again = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0.2,
                                           workspace=ws, rows_per_block=R)
    torch.cuda.synchronize()
    for key in ("loss", "divergence", "mask", "dHidden", "dW"):
        assert torch.equal(again[key], out[key]), key
    del again
    # four copies of the batch in one call: every row's outputs repeat, dW and the loss are those of one copy (the scale
    # is a quarter, added four times: exactly, since a power of two commutes with the roundings)
    rep = lambda x: x.repeat(4, *([1] * (x.dim() - 1))).contiguous()
    big = dppo.dppo_fused_lmhead_fwd_bwd(rep(b.hidden), b.lm_head, rep(b.sampled_ids), rep(b.mu_logp), rep(b.advantages), None,
                                         dppo.BINARY_TV, 0.2, workspace=ws, rows_per_block=R)
    torch.cuda.synchronize()
    assert int(big["status"].item()) == 0
    assert torch.equal(big["mask"], rep(out["mask"])) and torch.equal(big["divergence"], rep(out["divergence"]))
    assert torch.allclose(big["dHidden"], 0.25 * rep(out["dHidden"]), rtol=1e-6, atol=0)
    assert torch.allclose(big["dW"], out["dW"], rtol=2e-3, atol=1e-3 * float(out["dW"].abs().max().item()))
    assert abs(float(big["loss"].item()) - float(out["loss"].item())) <= 1e-5 * abs(float(out["loss"].item()))


def test_fused_full_size_topk_sampled_rows():
    """The fused configuration at full size with the Top-K TV divergence (K = 20): sampled rows against the oracle."""
    T, d, V, K = 8192, 2048, 151936, 20
    b = wl.lm_head_workload(DEV, seed=5, K=K)
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.TOPK_TV, 0.2,
                                         K=K, mu_topk_ids=b.mu_topk_ids, mu_topk_p=b.mu_topk_p)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    g = torch.Generator().manual_seed(10)
    rows = torch.sort(torch.randperm(T, generator=g)[:16]).values
    ridx = rows.numpy()
    W64 = b.lm_head.float().cpu().numpy().astype(np.float64)
    Hr = b.hidden[rows.to(DEV)].float().cpu().numpy().astype(np.float64)
    orr = O.dppo_fused_lmhead_fwd_bwd(Hr, W64, b.sampled_ids.cpu().numpy()[ridx], b.mu_logp.cpu().numpy().astype(np.float64)[ridx],
                                      b.advantages.cpu().numpy().astype(np.float64)[ridx], None, O.TOPK_TV, 0.2, 1.0 / T, K,
                                      b.mu_topk_ids.cpu().numpy()[ridx], b.mu_topk_p.cpu().numpy().astype(np.float64)[ridx])
    P.check_scalars(out["divergence"].cpu().numpy()[ridx], out["mask"].cpu().numpy()[ridx], orr, dict(token_mask=None), 0.2)
    eh = np.abs(out["dHidden"][rows.to(DEV)].cpu().numpy() - orr["dHidden"])
    assert np.all(eh <= 2.0 ** -8 * (np.abs(orr["dlogits"]) @ np.abs(W64).T) + 1e-7 * np.abs(orr["dHidden"]).max())
    assert torch.isfinite(out["dW"]).all()

