"""The entry points only enqueue work on the caller's stream (no allocation, no synchronisation), so a step can be
captured in a CUDA graph and replayed; small batches, where launch overhead dominates, are the use."""
import pytest
import torch

import paper_2602_04879_b200 as dppo
from paper_2602_04879_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_streaming_entry_point_replays_from_a_cuda_graph():
    b = wl.tiny_binary_tv(DEV, seed=0)
    dl = torch.empty_like(b.logits)
    ws = torch.empty(dppo.dppo_workspace_bytes(b.T), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    call = lambda: dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, 0, 0.2,
                                          dlogits=dl, workspace=ws, status=st)
    eager = call()
    torch.cuda.synchronize()
    ref = {k: eager[k].clone() for k in ("loss", "divergence", "mask", "dlogits")}
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        out = call()
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
