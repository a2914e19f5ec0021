"""The entry point for callers that cannot allocate device memory (collected last on purpose).

``dppo_loss_fwd_bwd_static_ws`` takes its scratch from an array built into the library instead of a
caller-provided workspace.  It is meant for code that has no way to obtain device memory at call time,
for example because a framework allocator already owns the whole GPU or because the step loop must not
hit the device-wide stall of cudaMalloc.  The test drives it through the C ABI twice in a row, with
different shapes, and compares each result with the regular entry point on the same inputs, using the
tolerances of the parity tests.
"""
import numpy as np
import pytest
import torch

import paper_2602_04879_b200 as dppo
from paper_2602_04879_b200 import binding
from paper_2602_04879_b200 import workloads as wl

DEV = "cuda:0"


def _compare(new, ref, bf16_out):
    torch.cuda.synchronize()
    assert int(new["status"].item()) == 0 and int(ref["status"].item()) == 0
    assert torch.equal(new["mask"], ref["mask"])
    dn, dr = new["divergence"].double().cpu().numpy(), ref["divergence"].double().cpu().numpy()
    assert np.array_equal(np.isfinite(dn), np.isfinite(dr))
    assert np.max(np.abs(dn[np.isfinite(dn)] - dr[np.isfinite(dr)])) <= 1e-5
    ln, lr = float(new["loss"].item()), float(ref["loss"].item())
    assert abs(ln - lr) <= 1e-4 * abs(lr) + 1e-12
    a, b = new["dlogits"].float(), ref["dlogits"].float()
    if bf16_out:
        assert torch.all((a - b).abs() <= 2.0 ** -7 * b.abs())          # at most one bf16 ulp apart
    else:
        assert (a - b).abs().max().item() <= 2e-3 * b.abs().max().item()


@pytest.mark.gpu
def test_static_scratch_entry_matches_regular_entry_twice():
    # first call: Qwen3-vocabulary rows, Top-K KL (exercises every per-row scratch column)
    b1 = wl.qwen_vocab_rows(DEV, seed=21, n_resp=5, resp_len=40, K=20, group=5)
    ref1 = dppo.dppo_loss_fwd_bwd(b1.logits, b1.sampled_ids, b1.mu_logp, b1.advantages, None, dppo.TOPK_KL, 20, 0.01,
                                  b1.mu_topk_ids, b1.mu_topk_p, want_stats=True)
    new1 = dppo.dppo_loss_fwd_bwd_static_ws(b1.logits, b1.sampled_ids, b1.mu_logp, b1.advantages, None, dppo.TOPK_KL, 20,
                                            0.01, b1.mu_topk_ids, b1.mu_topk_p)
    _compare(new1, ref1, bf16_out=True)
    # second call right after it: fewer rows, fp32 logits, a token mask; the array still holds call 1's rows
    b2 = wl.tiny_binary_tv(DEV, seed=22, T=96, V=4096)
    b2.token_mask = (torch.arange(96, device=DEV) % 5 != 0).to(torch.uint8)
    new2 = dppo.dppo_loss_fwd_bwd_static_ws(b2.logits, b2.sampled_ids, b2.mu_logp, b2.advantages, b2.token_mask,
                                            dppo.BINARY_KL, 0, 1e-4)
    ref2 = dppo.dppo_loss_fwd_bwd(b2.logits, b2.sampled_ids, b2.mu_logp, b2.advantages, b2.token_mask, dppo.BINARY_KL, 0, 1e-4)
    _compare(new2, ref2, bf16_out=False)
    # and call 1 again gives call 1's result again
    new3 = dppo.dppo_loss_fwd_bwd_static_ws(b1.logits, b1.sampled_ids, b1.mu_logp, b1.advantages, None, dppo.TOPK_KL, 20,
                                            0.01, b1.mu_topk_ids, b1.mu_topk_p)
    _compare(new3, ref1, bf16_out=True)


@pytest.mark.gpu
def test_static_scratch_entry_rejects_too_many_rows():
    T = binding.STATIC_WS_MAX_ROWS + 1
    logits = torch.zeros((T, 8), dtype=torch.bfloat16, device=DEV)
    ids = torch.zeros(T, dtype=torch.int32, device=DEV)
    f = torch.zeros(T, dtype=torch.float32, device=DEV)
    with pytest.raises(dppo.DppoError) as e:
        dppo.dppo_loss_fwd_bwd_static_ws(logits, ids, f, f)
    assert e.value.code == -12 and "DPPO_STATIC_WS_MAX_ROWS" in str(e.value)
