"""Data parallelism over token rows.

Rows of x are independent, so every rank runs the forward pass and dX on its own
rows with the (replicated) codes, qparams, A and B and exchanges nothing.  dA and
dB are sums over rows: one all-reduce (sum, fp32) of (G*r + r*N) values per layer
is the only exchange step.  torch.distributed carries it (NCCL between GPUs,
gloo on CPU in the tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(m: int, rank: int, world: int):
    """Contiguous, balanced slice [start, stop) of m token rows owned by `rank`."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the group")
    base, extra = divmod(m, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def allreduce_adapter_grads(dA: torch.Tensor, dB: torch.Tensor, group=None):
    """Sums the per-rank adapter gradients in place over the process group."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(dA, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(dB, op=dist.ReduceOp.SUM, group=group)
    return dA, dB
