"""The entry point for callers that cannot allocate device memory (collected last on purpose).

``dppo_loss_fwd_bwd_static_ws`` takes its scratch from an array built into the library instead of a
caller-provided workspace.  It is meant for code that has no way to obtain device memory at call time,
for example because a framework allocator already owns the whole GPU or because the step loop must not
hit the device-wide stall of cudaMalloc.  The test drives it through the C ABI three times in a row, with
different shapes, and holds each result to the float64 oracle with the tolerances of the parity tests
(and to the regular entry point, whose kernels it shares, bit for bit).
"""
import os
import re

import numpy as np
import pytest
import torch

import paper_2602_04879_b200 as dppo
from paper_2602_04879_b200 import binding
from paper_2602_04879_b200 import workloads as wl

import parity_util as P

DEV = "cuda:0"


def _check(new, batch, variant, K, delta, bf16_out, is_cap=0.0):
    torch.cuda.synchronize()
    assert int(new["status"].item()) == 0
    h = P.host_inputs(batch)
    ora = P.run_oracle(h, variant, K, delta, None, is_cap=is_cap if is_cap > 0 else None)
    P.check_scalars(new["divergence"].cpu().numpy(), new["mask"].cpu().numpy(), ora, h, delta)
    P.check_loss(float(new["loss"].item()), ora["loss"], batch.logits.dtype == torch.bfloat16, ora["row_loss"])
    P.check_dlogits(new["dlogits"], ora["dlogits"], out_is_bf16=bf16_out)
    ref = dppo.dppo_loss_fwd_bwd(batch.logits, batch.sampled_ids, batch.mu_logp, batch.advantages, batch.token_mask, variant, K, delta,
                                 batch.mu_topk_ids, batch.mu_topk_p, is_cap=is_cap)
    torch.cuda.synchronize()
    for key in ("loss", "divergence", "mask", "dlogits"):
        assert torch.equal(new[key], ref[key]), key


@pytest.mark.gpu
def test_static_scratch_entry_matches_the_oracle_on_calls_in_a_row():
    # first call: Qwen3-vocabulary rows, Top-K KL with an importance cap (exercises every per-row scratch column)
    b1 = wl.qwen_vocab_rows(DEV, seed=21, n_resp=5, resp_len=40, K=20, group=5)
    new1 = dppo.dppo_loss_fwd_bwd_static_ws(b1.logits, b1.sampled_ids, b1.mu_logp, b1.advantages, None, dppo.TOPK_KL, 20,
                                            0.01, b1.mu_topk_ids, b1.mu_topk_p, is_cap=1.02)
    _check(new1, b1, dppo.TOPK_KL, 20, 0.01, bf16_out=True, is_cap=1.02)
    # second call right after it: fewer rows, fp32 logits, a token mask; the array still holds call 1's rows
    b2 = wl.tiny_binary_tv(DEV, seed=22, T=96, V=4096)
    b2.token_mask = (torch.arange(96, device=DEV) % 5 != 0).to(torch.uint8)
    new2 = dppo.dppo_loss_fwd_bwd_static_ws(b2.logits, b2.sampled_ids, b2.mu_logp, b2.advantages, b2.token_mask,
                                            dppo.BINARY_KL, 0, 1e-4)
    _check(new2, b2, dppo.BINARY_KL, 0, 1e-4, bf16_out=False)
    # and call 1 again gives call 1's result again
    new3 = dppo.dppo_loss_fwd_bwd_static_ws(b1.logits, b1.sampled_ids, b1.mu_logp, b1.advantages, None, dppo.TOPK_KL, 20,
                                            0.01, b1.mu_topk_ids, b1.mu_topk_p, is_cap=1.02)
    _check(new3, b1, dppo.TOPK_KL, 20, 0.01, bf16_out=True, is_cap=1.02)
    for key in ("loss", "divergence", "mask", "dlogits"):
        assert torch.equal(new3[key], new1[key]), key


@pytest.mark.gpu
def test_static_scratch_entry_rejects_too_many_rows():
    T = binding.STATIC_WS_MAX_ROWS + 1
    logits = torch.zeros((T, 8), dtype=torch.bfloat16, device=DEV)
    ids = torch.zeros(T, dtype=torch.int32, device=DEV)
    f = torch.zeros(T, dtype=torch.float32, device=DEV)
    with pytest.raises(dppo.DppoError) as e:
        dppo.dppo_loss_fwd_bwd_static_ws(logits, ids, f, f)
    assert e.value.code == -12 and "DPPO_STATIC_WS_MAX_ROWS" in str(e.value)


def test_binding_repeats_the_header_limit():
    """The row limit of the built-in scratch array is a macro of the header; the binding's copy must be the same number."""
    hdr = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "dppo.h")).read()
    m = re.search(r"#define\s+DPPO_STATIC_WS_MAX_ROWS\s+(\d+)", hdr)
    assert m and int(m.group(1)) == binding.STATIC_WS_MAX_ROWS
