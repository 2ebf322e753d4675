"""Data-parallel plumbing of the DP-SGD step (torch.distributed; NCCL on GPUs, gloo in tests).

Examples are independent in every norm step and the clipped sum adds over examples, so the
batch shards across ranks with ONE exchange: the clipped sums are all-reduced, then every rank
adds the same noise stream (same seed, tensor id and step), which keeps replicas identical
without a broadcast.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence, Tuple

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


def bucket_order(linear_names: Sequence[str], head_name: Optional[str], table_names: Sequence[str],
                 n_linear_buckets: int = 3) -> List[List[str]]:
    """Order in which the clipped sums are produced AND exchanged: the LM head first (the largest
    tensor: its exchange then overlaps everything that follows), the block linears in
    `n_linear_buckets` contiguous groups, the embedding tables and small vectors last.  Every name
    appears exactly once; empty buckets are dropped."""
    buckets: List[List[str]] = []
    if head_name is not None:
        buckets.append([head_name])
    names = list(linear_names)
    k = max(1, min(n_linear_buckets, len(names))) if names else 0
    for b in range(k):
        lo, hi = shard_range(len(names), b, k)
        buckets.append(names[lo:hi])
    buckets.append(list(table_names))
    return [b for b in buckets if b]


class BucketedExchange:
    """Reduce-scatter of the clipped sums, bucket by bucket, on a communication stream.

    submit(names) is called right after the kernels that produce those tensors were enqueued on the
    compute stream: an event orders the bucket's collectives behind them, and the collectives (and
    the noise of the slice this rank owns) run on the communication stream while the compute
    stream goes on with the next bucket.  Nothing is ever enqueued on the compute stream; finish()
    makes it wait for the communication stream at the end of the step.

    After finish(), owned[name] = (begin, end, tensor) is this rank's slice of the summed, noised
    tensor; with gather=True the slices are also all-gathered back into `outs`.  Buffers are
    allocated once.  On CPU tensors (tests) there are no streams and everything runs in line.
    """

    def __init__(self, outs: Dict[str, torch.Tensor],
                 add_noise_slice: Callable[[torch.Tensor, int, int, object], None],
                 group=None, gather: bool = False):
        self.outs, self.group, self.gather = outs, group, gather
        self.add_noise_slice = add_noise_slice
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.tid = {name: t for t, name in enumerate(sorted(outs))}
        any_t = next(iter(outs.values()))
        self.cuda = any_t.is_cuda
        self.comm = torch.cuda.Stream(device=any_t.device) if self.cuda else None
        self.owned: Dict[str, Tuple[int, int, torch.Tensor]] = {}
        self._buf: Dict[str, Tuple[torch.Tensor, Optional[torch.Tensor]]] = {}
        self.submitted: List[str] = []
        self.bytes_on_wire = 0          # per rank and step: what this rank sends (and receives)
        for name, t in outs.items():
            flat = t.view(-1)
            chunk, lo, hi = slice_bounds(flat.numel(), self.rank, self.world)
            padded = None if chunk * self.world == flat.numel() else flat.new_zeros(chunk * self.world)
            own = torch.empty(chunk, dtype=flat.dtype, device=flat.device)
            self._buf[name] = (own, padded)
            self.owned[name] = (lo, hi, own[:max(hi - lo, 0)])
            frac = (self.world - 1) / self.world
            self.bytes_on_wire += int(chunk * self.world * flat.element_size() * frac * (2 if gather else 1))

    def begin_step(self) -> None:
        self.submitted = []
        if self.cuda:
            # the previous step's readers of the slices (optimizer, gather) are done
            self.comm.wait_stream(torch.cuda.current_stream())

    def submit(self, names: Sequence[str]) -> None:
        if self.cuda:
            ev = torch.cuda.Event()
            ev.record(torch.cuda.current_stream())
            self.comm.wait_event(ev)
            with torch.cuda.stream(self.comm):
                for name in names:
                    self._exchange(name, self.comm)
        else:
            for name in names:
                self._exchange(name, None)
        self.submitted.extend(names)

    def _exchange(self, name: str, stream) -> None:
        flat = self.outs[name].view(-1)
        numel = flat.numel()
        own, padded = self._buf[name]
        lo, hi, mine = self.owned[name]
        if self.world == 1:
            self.add_noise_slice(flat, 0, self.tid[name], stream)
            self.owned[name] = (0, numel, flat)
            return
        src = flat
        if padded is not None:
            padded[:numel].copy_(flat)
            src = padded
        dist.reduce_scatter_tensor(own, src, op=dist.ReduceOp.SUM, group=self.group)
        if hi > lo:
            self.add_noise_slice(mine, lo, self.tid[name], stream)
        if self.gather:
            dist.all_gather_into_tensor(src, own, group=self.group)
            if padded is not None:
                flat.copy_(padded[:numel])

    def finish(self) -> None:
        missing = set(self.outs) - set(self.submitted)
        if missing:
            raise RuntimeError(f"tensors never exchanged this step: {sorted(missing)}")
        if self.cuda:
            torch.cuda.current_stream().wait_stream(self.comm)
