"""Data-parallel plumbing for the compressed layer.

Tokens shard across ranks; Y, Z and dX are row-independent, W is replicated and
every rank regenerates the same P from (seed, layer, epoch), so the only exchange
of a step is the sum of the r x m compressed gradients Gc (Algorithm 2 line 1's
output) between the backward and the update.  One process drives one GPU.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys

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
    """Sums Gc (r x m, fp32) over the ranks in place; no-op without a process group.
    With the NCCL backend the collective is enqueued on the current stream, i.e. between
    the layer's backward and its update."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(Gc, op=dist.ReduceOp.SUM, group=group)
    return Gc


def layer_step(lay, X, dY, W, Y, Z, dX, Gc, M, V, group=None, lr=None) -> int:
    """One training step of one layer on this rank's token shard: Algorithm 1, Algorithm 2,
    the sum of Gc over the ranks, Algorithm 3, and the refresh check.  `lay` has the
    interface of binding.CompactLinear.  Returns the epoch the step ran under.  Every rank
    ends the step with the same W, M, V: the summed Gc is the same bits everywhere."""
    _, _, epoch = lay.forward(X, W, Y, Z)
    lay.backward(dY, Z, W, Gc, dX)
    allreduce_compressed_grad(Gc, group)
    if lr is None:
        lay.adam_update(W, Gc, M, V, epoch)
    else:
        lay.adam_update(W, Gc, M, V, epoch, lr=lr)
    lay.refresh_projection()
    return epoch


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def rank_launch_command(nproc: int, script: str, script_args, port: int | None = None):
    """The command that starts `nproc` ranks of `script` on this node, one per GPU, with
    RANK / LOCAL_RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT in each rank's environment."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
            "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), script, *script_args]


def spawn_ranks(nproc: int, script: str, script_args, port: int | None = None, env=None) -> int:
    """Runs `script` as `nproc` ranks and returns the launcher's exit code."""
    e = dict(os.environ if env is None else env)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        e.pop(k, None)
    return subprocess.call(rank_launch_command(nproc, script, list(script_args), port), env=e)
