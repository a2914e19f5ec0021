"""World-size-2 (and 3) checks of the row-sharding helpers on CPU with the gloo backend: shards cover every row once, the
global token-mean scale is agreed on, and the shards' losses (oracle per shard, global scale) add up to the oracle's
loss on the whole batch; gradient rows of a shard equal the corresponding rows of the whole-batch gradient."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_04879_b200 import parallel


def test_shard_rows_partition():
    for T in (0, 1, 5, 16, 17, 16384, 280294):
        for world in (1, 2, 3, 8):
            spans = [parallel.shard_rows(T, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    assert parallel.global_loss_scale(0) == 0.0 and parallel.global_loss_scale(4) == 0.25


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import dppo_oracle as O
        from paper_2602_04879_b200 import workloads as wl
        # the same seeded batch on every rank (T not divisible by the world size), ragged mask
        b = wl.qwen_vocab_rows("cpu", seed=31, n_resp=5, resp_len=7, V=512, K=6, group=5)
        T = b.T
        tok = (torch.arange(T) % 4 != 1).to(torch.uint8)
        z = b.logits.float().numpy().astype(np.float64)
        ids, mu, adv = b.sampled_ids.numpy(), b.mu_logp.numpy().astype(np.float64), b.advantages.numpy().astype(np.float64)
        tk_i, tk_p = b.mu_topk_ids.numpy(), b.mu_topk_p.numpy().astype(np.float64)
        lo, hi = parallel.shard_rows(T, rank, world)
        scale = parallel.global_loss_scale(tok[lo:hi])
        assert scale == 1.0 / int(tok.sum())
        part = O.dppo_loss_fwd_bwd(z[lo:hi], ids[lo:hi], mu[lo:hi], adv[lo:hi], tok[lo:hi].numpy(), O.TOPK_KL, 6, 0.01, scale,
                                   tk_i[lo:hi], tk_p[lo:hi])
        total = float(parallel.reduce_loss(torch.tensor(part["loss"], dtype=torch.float64)).item())
        full = O.dppo_loss_fwd_bwd(z, ids, mu, adv, tok.numpy(), O.TOPK_KL, 6, 0.01, None, tk_i, tk_p)
        assert abs(total - full["loss"]) <= 1e-12 * max(1.0, abs(full["loss"]))
        np.testing.assert_allclose(part["dlogits"], full["dlogits"][lo:hi], rtol=0, atol=1e-15)
        assert np.array_equal(part["M"], full["M"][lo:hi])
        # every rank saw a different, non-empty shard
        sizes = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(sizes, torch.tensor([hi - lo]))
        assert sum(int(s.item()) for s in sizes) == T
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_loss_matches_whole_batch(world, tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(world))
