"""Data-parallel plumbing for the compressed layer.

Tokens shard across ranks; Y, Z and dX are row-independent, W is replicated and
every rank regenerates the same P from (seed, layer, epoch), so the only exchange
of a step is the sum of the r x m compressed gradients Gc before the update.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(tokens: int, rank: int, world: int, multiple: int = 128) -> tuple[int, int]:
    """Contiguous [start, stop) token range of `rank`; shard sizes are multiples of
    `multiple` except possibly the last."""
    blocks = (tokens + multiple - 1) // multiple
    per, extra = divmod(blocks, world)
    b0 = rank * per + min(rank, extra)
    b1 = b0 + per + (1 if rank < extra else 0)
    return min(b0 * multiple, tokens), min(b1 * multiple, tokens)


def allreduce_compressed_grad(Gc: torch.Tensor, group=None) -> torch.Tensor:
    """Sums Gc (r x m, fp32) over the ranks in place; no-op without a process group."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(Gc, op=dist.ReduceOp.SUM, group=group)
    return Gc
