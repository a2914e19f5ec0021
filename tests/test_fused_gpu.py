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


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 256, 256), (300, 520, 200), (256, 1024, 1024), (1000, 264, 4104)])
def test_gemm_tn_bf16_matches_fp64_product(M, N, K):
    g = torch.Generator(device=DEV).manual_seed(M * 7 + N * 3 + K)
    A = torch.randn((M, K), generator=g, device=DEV).to(torch.bfloat16)
    B = torch.randn((N, K), generator=g, device=DEV).to(torch.bfloat16)
    C, status = dppo.dppo_gemm_tn_bf16(A, B)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = A.double().cpu().numpy() @ B.double().cpu().numpy().T          # exact bf16 products, float64 accumulation
    err = np.abs(C.cpu().numpy() - ref).max()
    assert err <= 2e-5 * np.abs(ref).max() + 1e-4, err
    # strided operands (views into wider buffers) and a strided output
    Aw = torch.zeros((M, K + 24), dtype=torch.bfloat16, device=DEV)
    Aw[:, :K] = A
    Cw = torch.full((M, N + 5), 7.0, dtype=torch.float32, device=DEV)
    dppo.dppo_gemm_tn_bf16(Aw[:, :K], B, C=Cw[:, :N])
    torch.cuda.synchronize()
    assert torch.equal(Cw[:, :N], C) and torch.all(Cw[:, N:] == 7.0)


def _fused_case(T, d, V, seed, resp_len):
    b = wl.lm_head_workload(DEV, seed=seed, T=T, d=d, V=V, resp_len=resp_len, sigma_w=0.02 * (2048 / d) ** 0.5)
    return b


def _check_fused(b, variant, delta, tok=None):
    out = dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, tok, variant, delta,
                                         want_stats=True)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    H = b.hidden.float().cpu().numpy().astype(np.float64)
    W = b.lm_head.float().cpu().numpy().astype(np.float64)
    tokh = None if tok is None else tok.cpu().numpy()
    ora = O.dppo_fused_lmhead_fwd_bwd(H, W, b.sampled_ids.cpu().numpy(), b.mu_logp.cpu().numpy().astype(np.float64),
                                      b.advantages.cpu().numpy().astype(np.float64), tokh, variant, delta)
    h = dict(token_mask=tokh)
    P.check_scalars(out["divergence"].cpu().numpy(), out["mask"].cpu().numpy(), ora, h, delta)
    P.check_loss(float(out["loss"].item()), ora["loss"], True, ora["row_loss"])
    # dlogits is rounded to bf16 before the two gradient GEMMs: |delta P| <= 2^-9 |P| entrywise, hence the entrywise bounds
    # 2^-8 (|P| |W|^T) and 2^-8 (|H|^T |P|) (factor 2 of slack for the fp32 arithmetic in front of the rounding)
    aP = np.abs(ora["dlogits"])
    bound_h = 2.0 ** -8 * (aP @ np.abs(W).T) + 1e-7 * np.abs(ora["dHidden"]).max()
    bound_w = 2.0 ** -8 * (np.abs(H).T @ aP) + 1e-7 * np.abs(ora["dW"]).max()
    eh = np.abs(out["dHidden"].cpu().numpy() - ora["dHidden"])
    ew = np.abs(out["dW"].cpu().numpy() - ora["dW"])
    assert np.all(eh <= bound_h), (eh / bound_h).max()
    assert np.all(ew <= bound_w), (ew / bound_w).max()
    # and in aggregate the error is far below the bound
    assert eh.max() <= 4e-3 * np.abs(ora["dHidden"]).max() and ew.max() <= 4e-3 * np.abs(ora["dW"]).max()
    return out, ora


@pytest.mark.parametrize("T,d,V", [(256, 128, 1024), (200, 72, 1000), (384, 256, 2304)])
def test_fused_matches_oracle_small(T, d, V):
    b = _fused_case(T, d, V, seed=41, resp_len=8)
    out, ora = _check_fused(b, dppo.BINARY_TV, 0.2)
    # mask stress near the median divergence, KL variant, ragged mask
    Dm = np.sort(ora["D"])
    delta = float(np.float32(0.5 * (Dm[len(Dm) // 2] + Dm[len(Dm) // 2 + 1])))
    tok = (torch.arange(T, device=DEV) % 7 != 3).to(torch.uint8)
    out2, ora2 = _check_fused(b, dppo.BINARY_TV, delta, tok)
    valid = tok.cpu().numpy() != 0
    assert 0 < int(((ora2["M"] == 0) & valid).sum()) < int(valid.sum())
    _check_fused(b, dppo.BINARY_KL, 1e-9, tok)


def test_fused_rejects_misuse():
    b = _fused_case(128, 64, 512, seed=42, resp_len=8)
    with pytest.raises(dppo.DppoError) as e:
        dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.TOPK_TV, 0.2)
    assert e.value.code == -4
    with pytest.raises(dppo.DppoError) as e:
        dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0.2,
                                       workspace=torch.empty(1024, dtype=torch.uint8, device=DEV))
    assert e.value.code == -8
