"""Data-parallel plumbing for the gated low-rank layer (one process per GPU).

The layer is token-wise, so it shards by tokens: the forward pass needs no
communication; the backward pass needs ONE sum over ranks of the weight
gradients dP, dQ and of dlog_alpha (dX stays local).  Every rank must use the
same Philox (seed, offset) so that the whole global batch shares one gate
sample (the paper shares the mask across the examples of a batch).  Only
`torch.distributed` collectives are used; nothing here touches peer memory.
"""
from __future__ import annotations

from typing import Iterable, Tuple

import torch
import torch.distributed as dist


def token_shard(T_global: int, rank: int, world: int) -> Tuple[int, int]:
    """(first token, number of tokens) of `rank` when T_global tokens are split as evenly as possible."""
    base, extra = divmod(T_global, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def gate_stream(step: int, seed: int = 0) -> Tuple[int, int]:
    """Philox (seed, offset) of training step `step`: a function of the step only, never of the rank."""
    return seed, step << 24


def allreduce_gradients(flat_buffers: Iterable[torch.Tensor], group=None) -> None:
    """Sum the given (flat, contiguous) gradient buffers over all ranks, in place."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    for buf in flat_buffers:
        dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
