"""Data parallelism over tokens for the L4Q linear layer (plumbing only).

The layer shards over tokens: weights and quantizer parameters are replicated,
every rank runs forward and backward on its own token batch, and the only
exchange is the sum of the parameter gradients dA, dB, ds, db.  That sum is
exact because the four gradients are linear in G = sum_t dY_t^T X_t (Eq. 11) and
the STE gate depends on the replicated weights only (Eq. 5-6, 13-14).  Y and dX
stay local to the rank that owns the tokens.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

PARAM_GRADS = ("dA", "dB", "ds", "db")


def token_shard(tokens: int, rank: int, world: int) -> slice:
    """Contiguous, balanced token range of one rank (ranks differ by at most one token)."""
    base, extra = divmod(tokens, world)
    start = rank * base + min(rank, extra)
    return slice(start, start + base + (1 if rank < extra else 0))


def allreduce_param_grads(grads: dict, group=None) -> None:
    """In-place sum over ranks of those of dA, dB, ds, db that `grads` holds (one all-reduce per tensor;
    a no-op for one rank)."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    for k in PARAM_GRADS:
        if k not in grads:
            continue
        dist.all_reduce(grads[k], op=dist.ReduceOp.SUM, group=group)
