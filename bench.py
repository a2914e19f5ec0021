"""Benchmark of the DPPO per-token loss path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one forward+backward pass of the whole path (prelude, row kernel, loss reduction) over one
batch of the Qwen3-vocabulary Binary-TV workload: T = 16384 token rows (16 responses x 1024), V = 151936,
bf16 logits and bf16 gradient, delta = 0.2, synthetic seeded inputs.  With N > 1 (launched by torchrun,
one process per GPU) every rank owns T rows of a global batch of N*T rows, with the global token-mean
scale passed in, so no collective is on the data path (weak scaling).  Rank 0 prints one JSON line.

`--impl reference` times the float64 CPU oracle instead (rank 0 only), a bounded sample of the same
workload per step.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

T_ROWS = 16384
VOCAB = 151936
DELTA = 0.2
METRIC = "tokens/sec fwd+bwd DPPO loss at V=151936 bf16"
BYTES_PER_TOKEN = 4 * VOCAB          # bf16 logits read (2V) + bf16 dlogits written (2V)
WORKLOAD = "qwen3_vocab_binary_tv: T=16384 (16 responses x 1024), V=151936, bf16 logits, Binary-TV, delta=0.2"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default="binary_tv", choices=["binary_tv", "binary_kl"])
    ap.add_argument("--rows", type=int, default=T_ROWS, help="rows per GPU; anything but the default is a reduced case for profiling, not the benchmark workload")
    ap.add_argument("--kernel", default="auto", choices=["auto", "ring", "generic"], help="row kernel of the main measurement")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--fused-only", action="store_true", help="run only the fused LM-head measurement (profiling aid)")
    ap.add_argument("--fused-rows", type=int, default=8192, help="token rows of the fused measurement; anything but 8192 is a reduced profiling case")
    ap.add_argument("--no-fused", action="store_true", help="skip the fused LM-head measurement (reported as an extra object at N=1)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the other streaming configurations and the exact-divergence monitor (extra objects at N=1)")
    ap.add_argument("--variants-only", action="store_true", help="run only those extra measurements (profiling aid)")
    ap.add_argument("--vocab-sweep", action="store_true",
                    help="run only the streaming kernel over other vocabulary sizes, with 1 and 2 SMs per row where rows are long (profiling aid)")
    return ap.parse_args()


# ----------------------------------------------------------------------------------------- peaks / clocks

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def measured_tensor_peak():
    """Sustained bf16 dense TFLOP/s (the fused step is a long back-to-back sequence of GEMMs)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json bf16_tflops_sustained)"
    return 1400.0, "fallback (about 1.4 PFLOP/s sustained, earlier measurement on this pool)"


def bench_fused(dppo, wl, dev, steps=40, warmup=10, T=8192):
    """Fused LM-head variant on its own workload: hidden [8192, 2048] x W [2048, 151936], Binary-TV, delta 0.2."""
    import torch
    d, V = 2048, VOCAB
    b = wl.lm_head_workload(dev, seed=5, T=T, d=d, V=V)
    ws = torch.empty(dppo.dppo_fused_workspace_bytes(T, d, V), dtype=torch.uint8, device=dev)
    dH = torch.empty((T, d), dtype=torch.float32, device=dev)
    dW = torch.empty((d, V), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def step():
        return dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None,
                                              dppo.BINARY_TV, DELTA, workspace=ws, dHidden=dH, dW=dW, status=status)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        out = step()
    e1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ms = e0.elapsed_time(e1) / steps
    # the same step when every fourth response carries zero advantage (all its samples scored alike): those rows have no
    # gradient and the backward GEMMs run over the remaining rows only
    adv_full = b.advantages
    resp = torch.arange(T, device=dev) // 512
    b.advantages = torch.where(resp % 4 == 3, torch.zeros_like(adv_full), adv_full)
    ms_sparse = _time_steps(torch, step, steps, warmup)          # same run length as above: the step is power-bound
    b.advantages = adv_full
    # the same step with the LM head (and its gradient) stored [V, d]
    w_vd = b.lm_head.t().contiguous()
    dW_vd = dW.view(V, d)
    fn_vd = lambda: dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, w_vd, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, DELTA,
                                                   workspace=ws, dHidden=dH, dW=dW_vd, status=status, w_is_vd=True)
    ms_vd = _time_steps(torch, fn_vd, steps, warmup)
    del w_vd
    # the same step with the Top-K TV divergence (K = 20): adds W^T and T x K gather dot products to the forward
    ms_topk = None
    if T == 8192:
        bk = wl.lm_head_workload(dev, seed=5, T=T, d=d, V=V, K=20)
        wsk = torch.empty(dppo.dppo_fused_workspace_bytes(T, d, V, 20), dtype=torch.uint8, device=dev)
        fn = lambda: dppo.dppo_fused_lmhead_fwd_bwd(bk.hidden, bk.lm_head, bk.sampled_ids, bk.mu_logp, bk.advantages, None,
                                                    dppo.TOPK_TV, DELTA, K=20, mu_topk_ids=bk.mu_topk_ids, mu_topk_p=bk.mu_topk_p,
                                                    workspace=wsk, dHidden=dH, dW=dW, status=status)
        ms_topk = _time_steps(torch, fn, steps, warmup)
        assert int(status.item()) == 0
        del bk, wsk
    # the same step finished in blocks of 2048 rows: the workspace is that of 2048 rows (0.7 GB instead of 2.6 GB)
    R = 2048
    ws_b = torch.empty(dppo.dppo_fused_workspace_bytes(min(T, R), d, V), dtype=torch.uint8, device=dev)
    fn_b = lambda: dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, DELTA,
                                                  workspace=ws_b, dHidden=dH, dW=dW, status=status, rows_per_block=R)
    ms_blocks = _time_steps(torch, fn_b, steps, warmup)
    ws_bytes, ws_b_bytes = ws.numel(), ws_b.numel()
    del ws_b
    # the two-pass mode (each logits tile computed twice, dW with one bf16 rounding instead of two)
    fn_2 = lambda: dppo.dppo_fused_lmhead_fwd_bwd(b.hidden, b.lm_head, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.BINARY_TV, DELTA,
                                                  workspace=ws, dHidden=dH, dW=dW, status=status, two_pass=True)
    ms_two_pass = _time_steps(torch, fn_2, steps, warmup)
    peak, src = measured_tensor_peak()
    useful = 6.0 * T * d * V / (ms * 1e-3) / 1e12          # forward + dHidden + dW; every logits tile is computed once
    return {"workload": ("" if T == 8192 else f"REDUCED to {T} rows (profiling case): ") + "fused_lm_head_binary_tv: hidden [8192,2048] bf16 x W [2048,151936] bf16, delta=0.2",
            "ms_per_step": ms, "tokens_per_s": T / (ms * 1e-3), "steps": steps, "warmup": warmup,
            "roofline": {"bound": "tensor", "achieved": useful, "peak": peak, "unit": "TFLOP/s", "frac": useful / peak,
                         "traffic": None, "peak_source": "of " + src,
                         "flop_count": "6*T*d*V (forward, dHidden, dW); nothing is recomputed"},
            "gpu_launches_per_step": 17, "loss": float(out["loss"].item()),
            "ms_per_step_quarter_of_responses_zero_advantage": ms_sparse, "ms_per_step_topk_tv_k20": ms_topk,
            "ms_per_step_lm_head_vocab_major": ms_vd,
            "ms_per_step_row_blocks_2048": ms_blocks, "ms_per_step_two_pass": ms_two_pass, "workspace_bytes": ws_bytes, "workspace_bytes_row_blocks_2048": ws_b_bytes}


def _time_steps(torch, fn, steps, warmup):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def bench_vocab_sweep(dppo, wl, dev, steps=100, warmup=10):
    """The streaming kernel at the vocabulary sizes of other model families (bf16, about 2.5 GB of logits each, Binary-TV
    and Top-K TV with K = 20): ms per launch and fraction of the measured HBM copy peak (bytes = logits read + dlogits
    written), with the automatic number of SMs per row and, for rows of 19 chunks of 16 KB and more, with 1 and 2 forced."""
    import torch
    peak, peak_src = measured_peaks()
    out = []
    for V in (32000, 32768, 50257, 65536, 128256, 151936, 155648, 180224, 201088, 221184, 262144):
        T = max(148, (2_500_000_000 // (V * 2)) // 148 * 148) // 4 * 4
        b = wl.qwen_vocab_rows(dev, seed=3, n_resp=4, resp_len=T // 4, V=V, K=20, group=4)
        dl = torch.empty_like(b.logits)
        ws = torch.empty(dppo.dppo_workspace_bytes(T), dtype=torch.uint8, device=dev)
        st = torch.zeros(1, dtype=torch.int32, device=dev)
        chunks = -(-V * 2 // 16384)
        for cl in ((0,) if chunks < 19 else (0, 1, 2)):
            row = {"V": V, "rows": T, "chunks_per_row": chunks, "row_cluster": cl}
            for name, var, K in (("binary_tv", dppo.BINARY_TV, 0), ("topk_tv_k20", dppo.TOPK_TV, 20)):
                fn = lambda: dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, var, K, DELTA, dlogits=dl, workspace=ws,
                                                    status=st, mu_topk_ids=b.mu_topk_ids if K else None, mu_topk_p=b.mu_topk_p if K else None,
                                                    row_cluster=cl)
                ms = _time_steps(torch, fn, steps, warmup)
                row[name] = {"ms": round(ms, 4), "frac_of_hbm_peak": round(T * V * 4 / (ms * 1e-3) / 1e9 / peak, 3)}
            assert int(st.item()) == 0
            out.append(row)
        del b, dl
    return {"peak_gbs": peak, "peak_source": "of " + peak_src, "cases": out}


def bench_other_configs(dppo, wl, dev, steps=100, warmup=10, n_resp=16):
    """The other streaming configurations at full size (same kernel, other variant switches), and the exact
    full-vocabulary divergence monitor.  Extra objects of the benchmark line; the headline stays Binary-TV."""
    import torch
    peak, src = measured_peaks()
    out = {}

    def entry(ms, rows, valid, bytes_moved, note):
        gbs = bytes_moved / (ms * 1e-3) / 1e9
        return {"ms_per_step": ms, "rows_per_s": rows / (ms * 1e-3), "valid_tokens_per_s": valid / (ms * 1e-3),
                "achieved_gbs": gbs, "frac_of_hbm_peak": gbs / peak, "peak_source": "of " + src, "note": note}

    # the tiny configuration (T = 256, V = 4096, fp32): latency of one call, L2 flushed between the timed calls
    tb = wl.tiny_binary_tv(dev, seed=0)
    tdl = torch.empty_like(tb.logits)
    tws = torch.empty(dppo.dppo_workspace_bytes(tb.T), dtype=torch.uint8, device=dev)
    tst = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    tiny = lambda: dppo.dppo_loss_fwd_bwd(tb.logits, tb.sampled_ids, tb.mu_logp, tb.advantages, None, dppo.BINARY_TV, 0, 0.2,
                                          dlogits=tdl, workspace=tws, status=tst)
    for _ in range(3):
        tiny()
    us = []
    for _ in range(20):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        tiny()
        e1.record()
        torch.cuda.synchronize()
        us.append(1e3 * e0.elapsed_time(e1))
    us.sort()
    # the same call captured in a CUDA graph and replayed back to back (no L2 flush): what launch overhead leaves
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        tiny()
    us_replay = 1e3 * _time_steps(torch, graph.replay, 200, 5)
    out["tiny_binary_tv_fp32"] = {"us_per_call_median": us[len(us) // 2], "us_per_call_best": us[0], "calls": len(us),
                                  "us_per_graph_replay": us_replay,
                                  "note": "T=256, V=4096, fp32, all valid, delta=0.2: three launches per call, 8.4 MB moved; "
                                          "latency-bound; a 256 MB buffer is written between the timed calls (L2 flush)"}
    del graph, flush, tb, tdl, tws
    # Binary-KL and Top-K TV (K = 20) on the Qwen3-vocabulary rows
    b = wl.qwen_vocab_rows(dev, seed=1, K=20, n_resp=n_resp, group=min(16, n_resp))     # n_resp != 16: reduced profiling case
    T = b.T
    dl = torch.empty_like(b.logits)
    ws = torch.empty(dppo.dppo_workspace_bytes(T), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for name, variant, K, delta in (("binary_kl_delta0.1", dppo.BINARY_KL, 0, 0.1), ("topk_tv_k20_delta0.2", dppo.TOPK_TV, 20, 0.2)):
        fn = lambda: dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, variant, K, delta,
                                            b.mu_topk_ids, b.mu_topk_p, dlogits=dl, workspace=ws, status=status)
        ms = _time_steps(torch, fn, steps, warmup)
        out[name] = entry(ms, T, T, T * BYTES_PER_TOKEN, f"T={T}, V=151936, bf16 in/out; bytes = logits read + dlogits written")
    # exact full-vocabulary TV / KL / entropy from the trainer's and the rollout's logits (two tensors read, nothing written)
    zmu = torch.empty_like(b.logits)
    g = torch.Generator(device=dev).manual_seed(77)
    for r0 in range(0, T, 1024):
        zmu[r0:r0 + 1024] = (b.logits[r0:r0 + 1024].float() + 0.1 * torch.randn((min(1024, T - r0), VOCAB), generator=g, device=dev)).to(torch.bfloat16)
    ms = _time_steps(torch, lambda: dppo.dppo_exact_divergence(b.logits, zmu, status=status), steps, warmup)
    out["exact_divergence"] = entry(ms, T, T, T * BYTES_PER_TOKEN, f"dppo_exact_divergence, T={T}, V=151936, bf16; bytes = both logits tensors read once "
                                    "(the second sweep is served by L2); 4 exp per element pair: the special-function pipe, not HBM, bounds it")
    # the monitor without the TV (tv = NULL): KL and entropy need one sweep, so each tensor is read once and nothing again
    ms1 = _time_steps(torch, lambda: dppo.dppo_exact_divergence(b.logits, zmu, status=status, want_tv=False), steps, warmup)
    out["exact_kl_only"] = entry(ms1, T, T, T * BYTES_PER_TOKEN, f"dppo_exact_divergence with tv = NULL (KL(mu||pi) and entropy only), T={T}, V=151936, bf16; "
                                 "bytes = both logits tensors read once; 2 exp per element pair")
    out["exact_kl_only"]["roofline"] = {"bound": "hbm", "achieved": out["exact_kl_only"]["achieved_gbs"], "peak": peak, "unit": "GB/s",
                                        "frac": out["exact_kl_only"]["frac_of_hbm_peak"], "peak_source": "of " + src}
    # DPPO with the exact KL as its trust region (the paper's delta_KL = 0.05): one-sweep monitor, then the loss kernel
    def exact_kl_then_loss():
        ex = dppo.dppo_exact_divergence(b.logits, zmu, status=status, want_tv=False)
        return dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.GIVEN_D, 0, 0.05,
                                      dlogits=dl, workspace=ws, status=status, given_divergence=ex["kl"])
    ms3 = _time_steps(torch, exact_kl_then_loss, steps, warmup)
    out["exact_kl_trust_region"] = entry(ms3, T, T, T * (BYTES_PER_TOKEN + 2 * VOCAB),
                                         f"dppo_exact_divergence(tv = NULL) + dppo_loss_fwd_bwd(GIVEN_D, delta 0.05), T={T}; bytes = both logits tensors read once + dlogits written")
    # DPPO with the exact TV as its trust region: the monitor, then the loss kernel on the divergence it produced
    def exact_then_loss():
        ex = dppo.dppo_exact_divergence(b.logits, zmu, status=status)
        return dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, dppo.GIVEN_D, 0, 0.2,
                                      dlogits=dl, workspace=ws, status=status, given_divergence=ex["tv"])
    ms2 = _time_steps(torch, exact_then_loss, steps, warmup)
    out["exact_tv_trust_region"] = entry(ms2, T, T, T * (BYTES_PER_TOKEN + 2 * VOCAB),
                                         f"dppo_exact_divergence + dppo_loss_fwd_bwd(GIVEN_D), T={T}; bytes = both logits tensors read once + dlogits written")
    # 4 ex2 per element pair on the special-function pipe (16 per clock and SM, 148 SMs, 1965 MHz maximum clock)
    sfu_peak = 148 * 16 * 1.965
    sfu = T * 4 * VOCAB / (ms * 1e-3) / 1e9
    out["exact_divergence"]["roofline"] = {"bound": "alu", "achieved": sfu, "peak": sfu_peak, "unit": "Gex2/s", "frac": sfu / sfu_peak,
                                           "peak_source": "148 SMs x 16 ex2/clk x 1.965 GHz (maximum SM clock)"}
    assert int(status.item()) == 0
    del b, dl, zmu
    torch.cuda.empty_cache()
    # Top-K KL, K = 64, ragged: two padded responses of the 64 (8192 rows each) with their token mask and the global scale
    lengths = wl.ragged_lengths()
    blocks = [wl.ragged_response(dev, i, lengths) for i in (0, 1)]
    cat = lambda xs: torch.cat(xs).contiguous()
    lg = cat([x.logits for x in blocks])
    for x in blocks:
        x.logits = None
    ids, mu, adv = cat([x.sampled_ids for x in blocks]), cat([x.mu_logp for x in blocks]), cat([x.advantages for x in blocks])
    tok, kid, kp = cat([x.token_mask for x in blocks]), cat([x.mu_topk_ids for x in blocks]), cat([x.mu_topk_p for x in blocks])
    T2, valid = lg.shape[0], int(tok.sum().item())
    dl = torch.empty_like(lg)
    ws = torch.empty(dppo.dppo_workspace_bytes(T2), dtype=torch.uint8, device=dev)
    scale = 1.0 / float(sum(lengths))
    fn = lambda: dppo.dppo_loss_fwd_bwd(lg, ids, mu, adv, tok, dppo.TOPK_KL, 64, 0.05, kid, kp, loss_scale=scale,
                                        dlogits=dl, workspace=ws, status=status)
    ms = _time_steps(torch, fn, steps, warmup)
    assert int(status.item()) == 0
    out["topk_kl_k64_ragged_delta0.05"] = entry(ms, T2, valid, valid * BYTES_PER_TOKEN + (T2 - valid) * 2 * VOCAB,
                                                f"responses 0 and 1 of the 64 as padded blocks of 8192 rows ({valid} valid of {T2}); "
                                                "bytes = valid rows read + every row of dlogits written (padding rows are zero-filled)")
    del lg, dl, blocks
    torch.cuda.empty_cache()
    if n_resp == 16:
        # the whole batch of 64 ragged responses (159 GB of padded logits: more than the device holds), streamed as 64 calls
        # of one padded block each with the global scale; each block is regenerated on the device (untimed), run once to
        # warm up and then timed over three calls; the batch time is the sum over the 64 blocks
        dl = torch.empty((8192, VOCAB), dtype=torch.bfloat16, device=dev)
        ws = torch.empty(dppo.dppo_workspace_bytes(8192), dtype=torch.uint8, device=dev)
        tot_ms, loss_sum = 0.0, 0.0
        for i in range(len(lengths)):
            x = wl.ragged_response(dev, i, lengths)
            fn = lambda: dppo.dppo_loss_fwd_bwd(x.logits, x.sampled_ids, x.mu_logp, x.advantages, x.token_mask, dppo.TOPK_KL, 64, 0.05,
                                                x.mu_topk_ids, x.mu_topk_p, loss_scale=scale, dlogits=dl, workspace=ws, status=status)
            tot_ms += _time_steps(torch, fn, 3, 1)
            loss_sum += float(fn()["loss"].item())
            del x
        assert int(status.item()) == 0
        nv, nrows = int(sum(lengths)), 8192 * len(lengths)
        e = entry(tot_ms, nrows, nv, nv * BYTES_PER_TOKEN + (nrows - nv) * 2 * VOCAB,
                  f"all 64 responses ({nv} valid of {nrows} padded rows), one call per padded block of 8192 rows, global scale 1/{nv}; "
                  "ms_per_step is the sum of the 64 calls; bytes = valid rows read + every row of dlogits written")
        e["loss"] = loss_sum
        e["calls"] = len(lengths)
        out["topk_kl_k64_ragged_whole_batch"] = e
    return out


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the row kernel.  Counted by ncu on the reduced
# case of the same kernel (T = 2048 rows, 1.2 GB on the device; mean of three launches: 696.1 MB read + 563.9 MB written
# for 622.3 + 622.3 MB algorithmic; summary under profiles/) and scaled to the T = 16384 rows of a benchmark launch: the
# traffic of this kernel is proportional to the rows it streams.  The reduced case flatters the writes a little (about
# 58 MB of the last rows are still dirty in L2 when the kernel ends).  Tied to the hash of the kernel sources: once they
# change the figure no longer applies and None is reported.
TRAFFIC_BYTES_PER_LAUNCH = int(round((696.08e6 + 563.85e6) * (T_ROWS / 2048)))
TRAFFIC_KERNEL_SHA = "587001d6fe5cd0f6"


def measured_traffic():
    import hashlib
    h = hashlib.sha256()
    for f in ("dppo_ring.cu", "dppo_common.cuh", "dppo_pipe.cuh", "dppo_rowtools.cuh"):
        with open(os.path.join(ROOT, "paper_2602_04879_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return TRAFFIC_BYTES_PER_LAUNCH if h.hexdigest()[:16] == TRAFFIC_KERNEL_SHA else None


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU from a thread (NVML) while the GPU works."""

    def __init__(self, index, uuid=None):
        self.samples = []
        self.stop_flag = False
        self.thread = None
        self.ok = False
        self.by = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            # NVML numbers the GPUs of the machine, CUDA those this process may see: resolve the handle from the CUDA
            # device's UUID, and fall back to the index only when that fails
            self.h = None
            if uuid:
                u = str(uuid)
                for cand in (u, "GPU-" + u, u.replace("GPU-", "")):
                    try:
                        self.h = pynvml.nvmlDeviceGetHandleByUUID(cand.encode() if hasattr(cand, "encode") else cand)
                        self.by = "uuid"
                        break
                    except Exception:  # noqa: BLE001
                        self.h = None
            if self.h is None:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
                self.by = "index"
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:  # noqa: BLE001
            self.max_mhz = None

    def _run(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                mem = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_MEM))
                try:
                    watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                except Exception:  # noqa: BLE001
                    watts = None
                self.samples.append((time.perf_counter(), mhz, reasons, mem, watts))
            except Exception:  # noqa: BLE001
                pass
            time.sleep(0.01)

    def start(self):
        self.stop_flag = False
        if self.ok:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()

    def stop(self):
        self.stop_flag = True
        if self.thread:
            self.thread.join(timeout=2)

    def summary(self, t0, t1):
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
                 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting"}
        sel = [s for s in self.samples if t0 <= s[0] <= t1] or self.samples
        if not sel:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "nvml_handle_by": self.by}
        mhz = sorted(s[1] for s in sel)
        bits = 0
        for s in sel:
            bits |= s[2]
        reasons = sorted(n for b, n in names.items() if bits & b)
        mem = sorted(s[3] for s in sel)
        watts = sorted(s[4] for s in sel if s[4] is not None)
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(sel),
                "mem_mhz": mem[len(mem) // 2], "power_w": watts[len(watts) // 2] if watts else None, "nvml_handle_by": self.by}


# ----------------------------------------------------------------------------------------- oracle arm

GEN_BLOCK = 512                      # rows per generator block of the workload (any block can be regenerated alone)
ORACLE_ROWS_PER_WORKER = 64


def host_cores():
    """Cores this process may use: the scheduler affinity, cut by a cgroup CPU quota if there is one."""
    try:
        n = len(os.sched_getaffinity(0))
    except AttributeError:
        n = os.cpu_count() or 1
    try:
        with open("/sys/fs/cgroup/cpu.max") as f:
            quota, period = f.read().split()
        if quota != "max":
            n = min(n, max(1, int(float(quota) / float(period))))
    except Exception:  # noqa: BLE001
        pass
    return max(1, n)


def oracle_workers():
    """One oracle process per host core, bounded so that the processes (an interpreter with torch and about 0.4 GB of
    float64 rows each) stay far inside the host's memory."""
    n = min(host_cores(), 96)
    try:
        with open("/proc/meminfo") as f:
            avail_kb = next(int(l.split()[1]) for l in f if l.startswith("MemAvailable"))
        n = min(n, max(1, int(avail_kb / 1048576 / 3)))
    except Exception:  # noqa: BLE001
        pass
    return max(1, n)


def _oracle_worker(w, seed, variant_code, iters, reps, barrier, queue):
    """One process of the CPU arm: regenerates its own 64 rows of the workload (untimed), then, `iters` times, meets the
    other workers at the barrier and runs the float64 oracle, as it stands, `reps` times over those rows."""
    try:
        import numpy as np
        import torch
        torch.set_num_threads(1)
        from paper_2602_04879_b200 import workloads as wl
        from oracle import dppo_oracle as O
        n = ORACLE_ROWS_PER_WORKER
        blocks = T_ROWS // GEN_BLOCK
        blk, m = w % blocks, (w // blocks) % (GEN_BLOCK // n)
        # a block is generated from its first row on: take the prefix that ends with this worker's rows
        b = wl.qwen_vocab_rows("cpu", seed=seed, row0=GEN_BLOCK * blk, rows=n * (m + 1))
        z = b.logits[n * m:].float().numpy().astype(np.float64)
        ids = b.sampled_ids[n * m:].numpy()
        mu = b.mu_logp[n * m:].numpy().astype(np.float64)
        adv = b.advantages[n * m:].numpy().astype(np.float64)
        del b
        for it in range(iters):
            barrier.wait(timeout=600)
            t0 = time.perf_counter()
            for _ in range(reps):
                O.dppo_loss_fwd_bwd(z, ids, mu, adv, None, variant_code, 0, DELTA, 1.0 / T_ROWS)
            queue.put((w, it, t0, time.perf_counter()))
    except Exception as e:  # noqa: BLE001
        queue.put((w, -1, repr(e), 0.0))


def oracle_parallel(seed, variant_code, iters, reps, workers=None):
    """Runs the oracle on `workers` processes at once (spawned: safe after CUDA has been initialised).  Returns per
    iteration the wall time from the first worker's start to the last worker's end (one monotonic clock for all
    processes of the machine), the rows processed per iteration, and the worker count."""
    import multiprocessing as mp
    W = workers or oracle_workers()
    ctx = mp.get_context("spawn")
    barrier, queue = ctx.Barrier(W), ctx.Queue()
    procs = [ctx.Process(target=_oracle_worker, args=(w, seed, variant_code, iters, reps, barrier, queue), daemon=True) for w in range(W)]
    for p in procs:
        p.start()
    spans = {}
    try:
        for _ in range(W * iters):
            w, it, t0, t1 = queue.get(timeout=1200)
            if it < 0:
                raise RuntimeError(f"oracle worker {w} failed: {t0}")
            lo, hi = spans.get(it, (t0, t1))
            spans[it] = (min(lo, t0), max(hi, t1))
    finally:
        for p in procs:
            p.join(timeout=30)
            if p.is_alive():
                p.kill()
    times = [spans[i][1] - spans[i][0] for i in range(iters)]
    return times, W * ORACLE_ROWS_PER_WORKER * reps, W


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import dppo_oracle as O
    code = O.BINARY_TV if args.variant == "binary_tv" else O.BINARY_KL
    steps = max(1, min(args.steps, 8))
    warm = max(0, min(args.warmup, 1))
    reps = 24                                     # 64 rows x 24 per worker and step: between one and two seconds of float64 numpy
    times, rows_per_step, W = oracle_parallel(1, code, warm + steps, reps)
    tot_t = sum(times[warm:])
    value = rows_per_step * steps / tot_t
    sample = (f"{W} processes (one per host core), each running the oracle {reps} times per step over its own "
              f"{ORACLE_ROWS_PER_WORKER} rows of the seeded batch = {rows_per_step} token rows per step; {steps} steps timed")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * tot_t / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "variant": args.variant, "note": "float64 numpy oracle on the host cores"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": W, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ----------------------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2602_04879_b200 as dppo
    from paper_2602_04879_b200 import parallel
    from paper_2602_04879_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    variant = dppo.BINARY_TV if args.variant == "binary_tv" else dppo.BINARY_KL
    if args.fused_only:
        print(json.dumps({"fused_lm_head": bench_fused(dppo, wl, dev, steps=max(1, min(args.steps, 40)), warmup=max(1, min(args.warmup, 10)), T=args.fused_rows)}))
        return

    if args.vocab_sweep:
        print(json.dumps({"vocab_sweep": bench_vocab_sweep(dppo, wl, dev, steps=max(1, min(args.steps, 100)), warmup=max(1, min(args.warmup, 10)))}))
        return

    if args.variants_only:
        print(json.dumps({"other_configs": bench_other_configs(dppo, wl, dev, steps=max(1, min(args.steps, 100)), warmup=max(1, min(args.warmup, 10)),
                                                                 n_resp=max(1, args.rows // 1024))}))
        return

    # each rank owns T rows of the global batch of world*T rows
    b = wl.qwen_vocab_rows(dev, seed=1 + rank, rows=args.rows) if args.rows != T_ROWS else wl.qwen_vocab_rows(dev, seed=1 + rank)
    T = b.T
    scale = parallel.global_loss_scale(T, device=dev)        # one all-reduce of N_valid, before the timed region
    dlogits = torch.empty_like(b.logits)
    ws = torch.empty(dppo.dppo_workspace_bytes(T), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    kernel_code = {"auto": dppo.KERNEL_AUTO, "ring": dppo.KERNEL_RING, "generic": dppo.KERNEL_GENERIC}[args.kernel]

    def step():
        return dppo.dppo_loss_fwd_bwd(b.logits, b.sampled_ids, b.mu_logp, b.advantages, None, variant, 0, DELTA,
                                      loss_scale=scale, dlogits=dlogits, workspace=ws, status=status, kernel=kernel_code)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    try:
        uuid = torch.cuda.get_device_properties(local).uuid
    except Exception:  # noqa: BLE001
        uuid = None
    sampler = ClockSampler(local, uuid)
    for _ in range(max(3, args.warmup)):
        out = step()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    t_host0 = time.perf_counter()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev0.record()
    marks[0].record()
    for i in range(args.steps):
        out = step()
        marks[i + 1].record()
    ev1.record()
    barrier()
    t_host1 = time.perf_counter()
    sampler.stop()
    ms = ev0.elapsed_time(ev1)
    if world > 1:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
        loss_val = float(parallel.reduce_loss(out["loss"]).item())   # global loss = sum of the shards' losses
    else:
        loss_val = float(out["loss"].item())
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    ms_per_step = ms / args.steps
    per_step = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps))       # this rank's steps, one by one
    tokens_per_s = world * T * args.steps / (ms * 1e-3)

    # roofline of the row kernel: algorithmic bytes of one launch over the step's device time (the step is
    # the row kernel plus two single-CTA kernels of a few microseconds, so this slightly under-reports it)
    peak, peak_src = measured_peaks()
    achieved = T * BYTES_PER_TOKEN / (ms_per_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None, "peak_source": "of " + peak_src, "kernel": "dppo_row_ring_kernel<bf16,bf16>",
                "algorithmic_bytes_per_launch": T * BYTES_PER_TOKEN}
    roofline["traffic"] = measured_traffic()
    clocks = sampler.summary(t_host0, t_host1)

    # the same step for a further stretch, long enough for the power management to settle (the timed region above is a
    # burst of some tens of milliseconds): what a training loop would see, with the clock it ran at
    sus_steps = max(200, args.steps)
    sus = ClockSampler(local, uuid)
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sus.start()
    th0 = time.perf_counter()
    s0.record()
    for _ in range(sus_steps):
        step()
    s1.record()
    barrier()
    th1 = time.perf_counter()
    sus.stop()
    sus_ms = s0.elapsed_time(s1) / sus_steps
    if world > 1:
        t = torch.tensor([sus_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        sus_ms = float(t.item())
    sc = sus.summary(th0, th1)
    sus_gbs = T * BYTES_PER_TOKEN / (sus_ms * 1e-3) / 1e9
    roofline["sustained"] = {"steps": sus_steps, "ms_per_step": sus_ms, "achieved": sus_gbs, "frac": sus_gbs / peak,
                             "sm_mhz": sc.get("sm_mhz"), "reasons": sc.get("reasons"), "power_w": sc.get("power_w"),
                             "ms_times_ghz": None if not sc.get("sm_mhz") else sus_ms * sc["sm_mhz"] / 1e3}
    assert int(status.item()) == 0

    line = {
        "metric": METRIC, "value": tokens_per_s, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD if T == T_ROWS else f"REDUCED to {T} rows (profiling case): " + WORKLOAD,
                   "variant": args.variant, "rows_per_gpu": T, "l2": "inputs_larger_than_L2 (4.98 GB read + 4.98 GB written per step)",
                   "parallelism": f"dp{world} row shards, no data-path collective", "logits_dtype": "bf16", "dlogits_dtype": "bf16"},
        "roofline": roofline, "clocks": clocks, "gpu_launches": 3 * args.steps, "loss": loss_val,
        "ms_per_step_best": per_step[0], "ms_per_step_median": per_step[len(per_step) // 2],
        "ms_times_ghz": None if not clocks.get("sm_mhz") else ms_per_step * clocks["sm_mhz"] / 1e3,
    }

    # end to end through the host-buffer entry point: pinned host inputs -> device -> loss, divergence, mask AND the
    # gradient back in pinned host memory (the gradient's copy back overlaps the next chunk's copy in)
    if not args.no_e2e:
        rows_per_chunk = 1024
        pin = lambda x: x.cpu().pin_memory()
        h = dict(logits=pin(b.logits), ids=pin(b.sampled_ids), mu=pin(b.mu_logp), adv=pin(b.advantages))
        outbuf = dict(divergence=torch.empty(T, dtype=torch.float32).pin_memory(), mask=torch.empty(T, dtype=torch.uint8).pin_memory(),
                      dlogits=torch.empty((T, VOCAB), dtype=torch.bfloat16).pin_memory())
        staging = torch.empty(dppo.dppo_host_staging_bytes(rows_per_chunk, VOCAB, 0, dppo.BF16), dtype=torch.uint8, device=dev)

        def e2e_step():
            return dppo.dppo_loss_fwd_bwd_host(h["logits"], h["ids"], h["mu"], h["adv"], None, variant, 0, DELTA,
                                               loss_scale=scale, rows_per_chunk=rows_per_chunk, staging=staging, out=outbuf,
                                               want_dlogits=True)
        e2e_steps = max(1, min(args.steps, 5))
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            r = e2e_step()                         # synchronises: results are on the host when it returns
        barrier()
        dt = time.perf_counter() - t0
        if world > 1:
            t = torch.tensor([dt], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            dt = float(t.item())
        assert r["status"] == 0
        # the gradient that arrived on the host is the one the device-resident step computed
        probe = [0, 1, T // 2, T - 1]
        same = bool(torch.equal(outbuf["dlogits"][probe], out["dlogits"][torch.as_tensor(probe, device=dev)].cpu()))
        line["e2e"] = {"gradient_on_host_equals_device_step": same,"value": world * T * e2e_steps / dt, "unit": "tokens/s",
                       "h2d_bytes_per_step": T * VOCAB * 2 + T * 12, "d2h_bytes_per_step": T * VOCAB * 2 + T * 5 + 8,
                       "steps": e2e_steps, "note": "dppo_loss_fwd_bwd_host: pinned host logits/ids/mu_logp/advantages in; loss, divergence, mask "
                                                   "and the bf16 gradient [T, V] out to pinned host memory"}
        del h, staging, outbuf

    if world == 1 and not args.no_fused and T == T_ROWS:
        del dlogits
        b.logits = None
        torch.cuda.empty_cache()
        line["fused_lm_head"] = bench_fused(dppo, wl, dev)
        if not args.no_variants:
            torch.cuda.empty_cache()
            line["other_configs"] = bench_other_configs(dppo, wl, dev)

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import dppo_oracle as O
        code = O.BINARY_TV if args.variant == "binary_tv" else O.BINARY_KL
        reps = 96                                 # 64 rows x 96 per process: several seconds of float64 numpy each
        times, rows, W = oracle_parallel(1, code, 1, reps)
        line["cpu_baseline"] = {"value": rows / times[0], "unit": "tokens/s", "cores": W, "kind": "oracle",
                                "sample": f"{W} processes (one per host core) each ran the float64 numpy oracle {reps} times over its own "
                                          f"{ORACLE_ROWS_PER_WORKER} rows of the workload, regenerated on the CPU: {rows} token rows in {times[0]:.1f} s"}
    if "fused_lm_head" in line:      # the tensor-bound variant's figures once more, compact, at the very end of the line
        f = line["fused_lm_head"]
        line["fused_summary"] = {"ms_per_step": f["ms_per_step"], "frac": f["roofline"]["frac"], "peak": f["roofline"]["peak"],
                                 "unit": "TFLOP/s", "achieved": f["roofline"]["achieved"], "steps": f["steps"],
                                 "ms_per_step_row_blocks": f.get("ms_per_step_row_blocks_2048")}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
