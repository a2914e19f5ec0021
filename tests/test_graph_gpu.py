"""The entry points only enqueue work on the caller's stream (no allocation, no synchronisation), so a step can be
captured in a CUDA graph and replayed; small batches, where launch overhead dominates, are the use."""
import pytest
import torch

import paper_2602_04879_b200 as dppo
from paper_2602_04879_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("row_cluster", [0, 2, 4])
def test_streaming_entry_point_replays_from_a_cuda_graph(row_cluster):
    """One SM per row, and rows shared by clusters of SMs (a cluster launch; for clusters of four the capture is the
    first use in this file, so the launcher's one-time query of how many clusters the device runs happens inside it)."""
    b = wl.tiny_binary_tv(DEV, seed=0)
    dl = torch.empty_like(b.logits)
    ws = torch.empty(dppo.dppo_workspace_bytes(b.T), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    call = lambda rc=row_cluster: dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0, 0.2,
                                                         dlogits=dl, workspace=ws, status=st, row_cluster=rc)
    eager = call(2 if row_cluster == 4 else row_cluster)      # same results up to the order of additions in the row sums
    torch.cuda.synchronize()
    ref = {k: eager[k].clone() for k in ("loss", "divergence", "mask", "dlogits")}
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        out = call()
    if row_cluster == 4:
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out["mask"], ref["mask"]) and torch.allclose(out["divergence"], ref["divergence"], atol=2e-6, rtol=0)
        assert torch.allclose(out["dlogits"], ref["dlogits"], rtol=1e-4, atol=1e-9) and int(st.item()) == 0
        ref = {k: out[k].clone() for k in ref}
    for _ in range(3):
        dl.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert all(torch.equal(out[k], ref[k]) for k in ref) and int(st.item()) == 0
    # new inputs in the captured buffers are picked up by the next replay
    b.advantages.neg_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out["loss"], -ref["loss"]) or abs(float(out["loss"].item()) + float(ref["loss"].item())) < 1e-6


def test_fused_entry_point_replays_from_a_cuda_graph():
    f = wl.lm_head_workload(DEV, seed=8, T=256, d=128, V=1024, resp_len=8, sigma_w=0.08)
    ws = torch.empty(dppo.dppo_fused_workspace_bytes(256, 128, 1024), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    call = lambda: dppo.dppo_fused_lmhead_fwd_bwd(f.hidden, f.lm_head, f.sampled_ids, f.mu_logp, f.advantages, None, dppo.BINARY_TV, 0.2,
                                                  workspace=ws, status=st)
    eager = call()
    torch.cuda.synchronize()
    ref = {k: eager[k].clone() for k in ("loss", "mask", "dHidden", "dW")}
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        out = call()
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    assert all(torch.equal(out[k], ref[k]) for k in ref) and int(st.item()) == 0
