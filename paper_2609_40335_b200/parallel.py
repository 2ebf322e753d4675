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


def slice_bounds(numel: int, rank: int, world: int) -> Tuple[int, int, int]:
    """(chunk, begin, end): rank's slice of a flat tensor split into `world` chunks whose length
    is a multiple of 4, so that every slice owns whole counters of the noise generator."""
    chunk = -(-numel // world)
    chunk = (chunk + 3) // 4 * 4
    begin = min(numel, rank * chunk)
    return chunk, begin, min(numel, begin + chunk)


def reduce_scatter_then_noise(outs: Dict[str, torch.Tensor],
                              add_noise_slice: Callable[[torch.Tensor, int, int], None],
                              group=None, gather: bool = True) -> Dict[str, Tuple[int, int, torch.Tensor]]:
    """The exchange as reduce-scatter: each rank receives the sum of ONE slice of every tensor,
    draws the noise of exactly that slice (`add_noise_slice(slice, first_element, tensor_id)`; the
    stream is indexed by element, so the result equals the single-process draw), and, with
    gather=True, the noised slices are all-gathered back into `outs` on every rank.  The noise
    work per rank is 1/world of the all-reduce form.  Returns {name: (begin, end, own slice)}.
    Tensors must be contiguous."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    owned = {}
    for tid, name in enumerate(sorted(outs)):
        flat = outs[name].view(-1)
        numel = flat.numel()
        if world == 1:
            add_noise_slice(flat, 0, tid)
            owned[name] = (0, numel, flat)
            continue
        chunk, lo, hi = slice_bounds(numel, rank, world)
        if chunk * world == numel:
            buf = flat
        else:                                   # pad to equal chunks
            buf = flat.new_zeros(chunk * world)
            buf[:numel].copy_(flat)
        own = torch.empty(chunk, dtype=flat.dtype, device=flat.device)
        dist.reduce_scatter_tensor(own, buf, op=dist.ReduceOp.SUM, group=group)
        if hi > lo:
            add_noise_slice(own[:hi - lo], lo, tid)
        owned[name] = (lo, hi, own[:hi - lo])
        if gather:
            dist.all_gather_into_tensor(buf, own, group=group)
            if buf is not flat:
                flat.copy_(buf[:numel])
    return owned
