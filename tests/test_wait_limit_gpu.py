"""The give-up path of the bounded on-chip waits.

Every wait inside the kernels (for a bulk copy to land, for another warp's result) has a time limit, after which the
CTA raises DPPO_STATUS_WAIT_LIMIT, stops touching memory and returns, so that a lost copy costs a call and not the GPU.
Here the limit is made to run out on purpose, in the one form that leaves nothing in flight: with
``test_inject = DPPO_INJECT_NO_COPIES`` the copy producers issue nothing, so the consumers wait for data that never
comes until ``wait_limit_us`` is over.  Nothing faults or hangs; the call returns, the status word carries the bit, and
an ordinary call right afterwards must match the oracle.
"""
import time

import numpy as np
import pytest
import torch

import paper_2602_04879_b200 as dppo
from paper_2602_04879_b200 import binding
from paper_2602_04879_b200 import workloads as wl
from oracle import dppo_oracle as O

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
LIMIT_US = 20000            # 20 ms per wait


def _small():
    return wl.tiny_binary_tv(DEV, seed=3, T=48, V=4096)


@pytest.mark.parametrize("row_cluster", [1, 2])
def test_row_kernel_gives_up_and_the_next_call_is_fine(row_cluster):
    """One SM per row, and pairs of SMs sharing the rows (they leave through their cluster barrier)."""
    b = _small()
    t0 = time.perf_counter()
    out = dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0, 0.2, row_cluster=row_cluster,
                                 kernel=dppo.KERNEL_RING, wait_limit_us=LIMIT_US, test_inject=binding.INJECT_NO_COPIES)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0                                   # a few waits of 20 ms, not the default 2 s each
    assert int(out["status"].item()) & binding.STATUS_WAIT_LIMIT
    # the same call without the injection, with the same short limit: waits take microseconds, so it never runs out
    out = dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0, 0.2, row_cluster=row_cluster,
                                 kernel=dppo.KERNEL_RING, wait_limit_us=LIMIT_US)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    h = P.host_inputs(b)
    ora = P.run_oracle(h, O.BINARY_TV, 0, 0.2, None)
    P.check_scalars(out["divergence"].cpu().numpy(), out["mask"].cpu().numpy(), ora, h, 0.2)
    P.check_loss(float(out["loss"].item()), ora["loss"], False, ora["row_loss"])
    P.check_dlogits(out["dlogits"], ora["dlogits"], out_is_bf16=False)


def test_exact_divergence_kernel_gives_up_and_the_next_call_is_fine():
    g = torch.Generator(device=DEV).manual_seed(5)
    z = 3.0 * torch.randn((40, 4096), generator=g, device=DEV)
    zm = z + 0.3 * torch.randn((40, 4096), generator=g, device=DEV)
    for want_tv in (True, False):
        out = dppo.dppo_exact_divergence(z, zm, want_tv=want_tv, wait_limit_us=LIMIT_US, test_inject=binding.INJECT_NO_COPIES)
        torch.cuda.synchronize()
        assert int(out["status"].item()) & binding.STATUS_WAIT_LIMIT
        out = dppo.dppo_exact_divergence(z, zm, want_tv=want_tv, wait_limit_us=LIMIT_US)
        torch.cuda.synchronize()
        assert int(out["status"].item()) == 0
        for t in (0, 17, 39):
            tv, kl, ent = O.exact_divergence_row(z[t].double().cpu().numpy(), zm[t].double().cpu().numpy())
            assert abs(out["kl"][t].item() - kl) <= 1e-5 and abs(out["entropy"][t].item() - ent) <= 2e-5 * max(1.0, ent)
            assert not want_tv or abs(out["tv"][t].item() - tv) <= 1e-5


@pytest.mark.parametrize("cta_group", [1, 2])
def test_tensor_core_gemm_gives_up_and_the_next_call_is_fine(cta_group):
    """Single SMs first, then pairs: with no copy issued no tensor-core instruction is issued either, every role of
    both CTAs of a pair runs into its own limit, the pair meets at its cluster barrier and frees its tensor memory."""
    g = torch.Generator(device=DEV).manual_seed(7)
    A = torch.randn((300, 200), generator=g, device=DEV).to(torch.bfloat16)
    B = torch.randn((520, 200), generator=g, device=DEV).to(torch.bfloat16)
    C, status = dppo.dppo_gemm_tn_bf16(A, B, cta_group=cta_group, wait_limit_us=LIMIT_US, test_inject=binding.INJECT_NO_COPIES)
    torch.cuda.synchronize()
    assert int(status.item()) & binding.STATUS_WAIT_LIMIT
    C, status = dppo.dppo_gemm_tn_bf16(A, B, cta_group=cta_group, wait_limit_us=LIMIT_US)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = A.double().cpu().numpy() @ B.double().cpu().numpy().T
    assert np.abs(C.cpu().numpy() - ref).max() <= 2e-5 * np.abs(ref).max() + 1e-4
