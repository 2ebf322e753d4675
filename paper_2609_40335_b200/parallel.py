"""Data-parallel plumbing of the DP-SGD step (torch.distributed; NCCL on GPUs, gloo in tests).

Examples are independent in every norm step and the clipped sum adds over examples, so the
batch shards across ranks with ONE exchange: the clipped sums are all-reduced, then every rank
adds the same noise stream (same seed, tensor id and step), which keeps replicas identical
without a broadcast.
"""
from __future__ import annotations

from typing import Callable, Dict, Tuple

import torch
import torch.distributed as dist


def shard_range(n_examples: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced [begin, end) slice of a global batch for one rank."""
    base, extra = divmod(n_examples, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def reduce_clipped_sums(outs: Dict[str, torch.Tensor], group=None) -> None:
    """Sum every clipped-sum tensor over ranks, in sorted key order on all ranks."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    for name in sorted(outs):
        dist.all_reduce(outs[name], op=dist.ReduceOp.SUM, group=group)


def reduce_then_noise(outs: Dict[str, torch.Tensor], add_noise: Callable[[torch.Tensor, int], None],
                      group=None) -> None:
    """The exchange step followed by one noise draw per tensor (tensor id = sorted position)."""
    reduce_clipped_sums(outs, group)
    for tid, name in enumerate(sorted(outs)):
        add_noise(outs[name], tid)
