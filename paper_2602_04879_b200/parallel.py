"""Host-side helpers for running the DPPO loss path data-parallel over token rows.

Rows are independent, so T rows are split into contiguous shards, one per rank.  The only
cross-rank quantities are two scalars: N_valid (needed *before* the call, because the
token-mean scale s = 1/N_valid enters every gradient row) and the loss (a sum of the shards'
losses *after* the call).  Both go through ``torch.distributed`` (NCCL on GPUs, gloo on CPU);
nothing else of the path communicates.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(T, rank, world):
    """Contiguous, balanced shard [start, stop) of T rows for ``rank`` of ``world``."""
    assert 0 <= rank < world and T >= 0
    base, rem = divmod(int(T), int(world))
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)


def global_loss_scale(n_valid_local, group=None, device=None):
    """Token-mean scale 1 / (sum over ranks of the local valid-row counts); 0.0 if no row is valid.
    ``n_valid_local`` is an int or a token-mask tensor of this rank's shard (None rows count as valid
    must be passed as an int)."""
    if torch.is_tensor(n_valid_local):
        device = n_valid_local.device if device is None else device
        n = (n_valid_local != 0).sum().to(torch.int64).reshape(1)
    else:
        n = torch.tensor([int(n_valid_local)], dtype=torch.int64, device=device or "cpu")
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(n, op=dist.ReduceOp.SUM, group=group)
    total = int(n.item())
    return (1.0 / total) if total > 0 else 0.0


def reduce_loss(loss_local, group=None):
    """Sum of the shards' losses (each computed with the global scale) = loss of the whole batch."""
    t = loss_local.detach().clone().reshape(1) if torch.is_tensor(loss_local) else torch.tensor([float(loss_local)], dtype=torch.float64)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t
