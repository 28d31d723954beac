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


def alloc_grad_bucket(shapes: dict, device="cpu", dtype=torch.float32):
    """One contiguous buffer holding the parameter gradients of a layer, and views of it by name.

    `shapes`: {name: shape} for the gradients to exchange (dA, dB, ds, db, or a subset).  Every view starts on
    a 16-byte boundary, as the library asks of its outputs.  Returns (flat, views); the kernels write the
    views, and one all-reduce of `flat` sums them all (the padding between views is zero and stays zero)."""
    offs, total = {}, 0
    for k in PARAM_GRADS:
        if k in shapes:
            offs[k] = total
            n = 1
            for d in shapes[k]:
                n *= int(d)
            total += (n + 3) // 4 * 4
    flat = torch.zeros(max(total, 4), dtype=dtype, device=device)
    views = {}
    for k, o in offs.items():
        n = 1
        for d in shapes[k]:
            n *= int(d)
        views[k] = flat[o:o + n].view(*shapes[k])
    return flat, views


def allreduce_grad_bucket(flat: torch.Tensor, group=None) -> None:
    """In-place sum over ranks of a bucket from alloc_grad_bucket: one collective per layer instead of one per
    tensor (these gradients are a few MB, so the collective's latency is what costs).  A no-op for one rank."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)


def allreduce_param_grads(grads: dict, group=None) -> None:
    """In-place sum over ranks of those of dA, dB, ds, db that `grads` holds (one all-reduce per tensor;
    a no-op for one rank)."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    for k in PARAM_GRADS:
        if k not in grads:
            continue
        dist.all_reduce(grads[k], op=dist.ReduceOp.SUM, group=group)
