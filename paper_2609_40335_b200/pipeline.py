"""One DP-SGD clipping step as a sequence of library calls (no arithmetic of its own).

Order (all enqueued on the current stream, no host synchronisation):
  norms of the block linears and the LM head  -> dp_ghost_norms          (Eq. 4 - Eq. 6)
  norm of the token (and position) embedding  -> dp_embed_norms
  tied head: cross term                       -> dp_tied_cross_term      (Eq. 11, Eq. 13)
  clipped sums per parameter tensor           -> dp_clip_accumulate[_embed]  (Eq. 2, Eq. 3, Eq. 7)
  Gaussian noise per parameter tensor         -> dp_add_noise            (Eq. 3)
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as dp
from .workloads import HostTensor, Workload

WPE_ROWS = 1024      # GPT-2's learned position table


def to_device(ht: HostTensor, device="cuda") -> torch.Tensor:
    """Upload a host tensor in its storage type (bf16 bit patterns are reinterpreted, not converted)."""
    if ht.dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(ht.data)).to(device)
    return torch.from_numpy(np.ascontiguousarray(ht.data).view(np.int16)).to(device).view(torch.bfloat16)


@dataclass
class DeviceStep:
    """Device-resident inputs, outputs and scratch of one step."""
    B: int
    T: int
    V: int
    C: float
    sigma: float
    tied: bool
    positions: bool
    linears: List[dp.Linear]
    lm: Optional[dp.Linear]
    ids: torch.Tensor
    pos_ids: Optional[torch.Tensor]
    G_emb: torch.Tensor
    d_model: int
    sq: torch.Tensor
    clip: torch.Tensor
    norms: torch.Tensor
    cross: Optional[torch.Tensor]
    dev_status: torch.Tensor
    outs: Dict[str, torch.Tensor] = field(default_factory=dict)
    vectors: List[dp.Vector] = field(default_factory=list)      # biases / LayerNorm parameters
    ws: Optional[torch.Tensor] = None
    side_stream: Optional[torch.cuda.Stream] = None     # work that overlaps the big norm kernel
    side: Optional[dict] = None       # side-stream buffers: own workspace, norm accumulator, sorts

    def input_bytes(self) -> int:
        """Bytes of input one step reads (a tensor shared by several layers counts every time)."""
        n = self.ids.numel() * 4 + self.G_emb.numel() * self.G_emb.element_size()
        for l in self.linears + ([self.lm] if self.lm else []):
            n += l.A.numel() * l.A.element_size() + l.G.numel() * l.G.element_size()
        return n


def upload(w: Workload, device="cuda", share_by_identity: bool = True) -> DeviceStep:
    cache = {}

    def up(ht):
        key = id(ht.data)
        if share_by_identity and key in cache:
            return cache[key]
        t = to_device(ht, device)
        cache[key] = t
        return t

    linears = [dp.Linear(up(l.A), up(l.G), d=l.d, p=l.p) for l in w.linears]
    lm = dp.Linear(up(w.lm.A), up(w.lm.G), d=w.lm.d, p=w.lm.p) if w.lm is not None else None
    ids = torch.from_numpy(w.ids).to(device)
    pos = None
    if w.positions:
        pos = torch.arange(w.T, dtype=torch.int32, device=device).repeat(w.B, 1).contiguous()
    ds = DeviceStep(
        B=w.B, T=w.T, V=w.V, C=w.C, sigma=w.sigma, tied=w.tied, positions=w.positions,
        linears=linears, lm=lm, ids=ids, pos_ids=pos, G_emb=up(w.G_emb), d_model=w.d_model,
        sq=torch.zeros(w.B, dtype=torch.float32, device=device),
        clip=torch.zeros(w.B, dtype=torch.float32, device=device),
        norms=torch.zeros(w.B, dtype=torch.float32, device=device),
        cross=torch.zeros(w.B, dtype=torch.float32, device=device) if w.tied else None,
        dev_status=torch.zeros(1, dtype=torch.int32, device=device))
    ds.vectors = [dp.Vector(up(v.G), up(v.X) if v.X is not None else None, p=v.p) for v in w.vectors]
    allocate(ds)
    return ds


def synthesize_on_device(name: str, B: int, T: int, d_model: int, n_blocks: int, V: int = 50257,
                         tied: bool = False, positions: bool = False, C: float = 1.0,
                         sigma: float = 1.0, seed: int = 0, device="cuda") -> DeviceStep:
    """Benchmark-only inputs drawn on the device (torch generator), for shapes whose host-side
    generation would take minutes: A ~ N(0,1), G ~ N(0,1e-4), Zipf(1.1) token ids, one tensor set
    per distinct layer shape shared by all blocks, LM-head pitch padded to a multiple of 8."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)

    def normal(rows, cols, std, ld=None):
        ld = ld or cols
        t = torch.empty(B, rows, ld, dtype=torch.bfloat16, device=device)
        step = max(1, (1 << 28) // (rows * ld))          # bounded fp32 staging buffer
        for b0 in range(0, B, step):
            b1 = min(B, b0 + step)
            x = torch.randn(b1 - b0, rows, ld, generator=g, device=device, dtype=torch.float32)
            t[b0:b1] = (x * std).to(torch.bfloat16)
        return t

    shapes = [(d_model, 3 * d_model), (d_model, d_model), (d_model, 4 * d_model), (4 * d_model, d_model)]
    sets = [(normal(T, d, 1.0), normal(T, p, 1e-2)) for d, p in shapes]
    linears = [dp.Linear(sets[k][0], sets[k][1], d=shapes[k][0], p=shapes[k][1])
               for _ in range(n_blocks) for k in range(4)]
    ldv = (V + 7) // 8 * 8
    lm = dp.Linear(normal(T, d_model, 1.0), normal(T, V, 1e-2, ld=ldv), d=d_model, p=V)
    w = torch.arange(1, V + 1, device=device, dtype=torch.float64) ** -1.1
    ids = torch.multinomial(w / w.sum(), B * T, replacement=True, generator=g).to(torch.int32).view(B, T)
    pos = torch.arange(T, dtype=torch.int32, device=device).repeat(B, 1).contiguous() if positions else None
    ds = DeviceStep(
        B=B, T=T, V=V, C=C, sigma=sigma, tied=tied, positions=positions, linears=linears, lm=lm,
        ids=ids, pos_ids=pos, G_emb=normal(T, d_model, 1e-2), d_model=d_model,
        sq=torch.zeros(B, dtype=torch.float32, device=device),
        clip=torch.zeros(B, dtype=torch.float32, device=device),
        norms=torch.zeros(B, dtype=torch.float32, device=device),
        cross=torch.zeros(B, dtype=torch.float32, device=device) if tied else None,
        dev_status=torch.zeros(1, dtype=torch.int32, device=device))
    allocate(ds)
    return ds


def allocate(ds: DeviceStep) -> None:
    """Output tensors (one per parameter tensor) and one workspace large enough for every call."""
    dev = ds.sq.device
    f32 = dict(dtype=torch.float32, device=dev)
    for k, l in enumerate(ds.linears):
        ds.outs[f"linear{k}"] = torch.empty(l.p, l.d, **f32)
    ds.outs["wte"] = torch.empty(ds.V, ds.d_model, **f32)
    if ds.lm is not None and not ds.tied:
        ds.outs["lm_head"] = torch.empty(ds.lm.p, ds.lm.d, **f32)
    if ds.positions:
        ds.outs["wpe"] = torch.empty(WPE_ROWS, ds.d_model, **f32)
    for k, v in enumerate(ds.vectors):
        ds.outs[f"vector{k}"] = torch.empty(v.p, **f32)
    every = ds.linears + ([ds.lm] if ds.lm else [])
    dt = dp._dt(every[0].A) if every else dp._dt(ds.G_emb)
    need = 256
    if every:
        need = max(need, dp.dp_ghost_norms_ws_bytes(every, ds.B, ds.T))
        need = max(need, dp.dp_clip_accumulate_grouped_ws_bytes(every, ds.B, ds.T))
    if ds.vectors:
        need = max(need, dp.dp_vector_norms_ws_bytes(ds.vectors, ds.B, ds.T))
        need = max(need, dp.dp_clip_accumulate_vectors_ws_bytes(ds.vectors, ds.B, ds.T))
    L = dp.load()
    need = max(need, int(L.dp_embed_norms_ws_bytes(ds.B, ds.T, ds.d_model)))
    need = max(need, int(L.dp_clip_accumulate_embed_ws_bytes(ds.B, ds.T, ds.d_model, ds.V)))
    if ds.positions:
        need = max(need, int(L.dp_clip_accumulate_embed_ws_bytes(ds.B, ds.T, ds.d_model, WPE_ROWS)))
    if ds.tied:
        need = max(need, int(L.dp_tied_cross_term_ws_bytes(ds.B, ds.T, ds.d_model, ds.V)))
    ds.ws = torch.empty(need, dtype=torch.uint8, device=dev)


def norms_phase(ds: DeviceStep, stream=None, after_first_launch=None) -> None:
    """Per-example squared norms into ds.sq (zeroed first), then norms and clip factors.
    after_first_launch: called right after the big norm kernel has been enqueued (used to start
    side-stream work that should share the SMs with it rather than run ahead of it)."""
    ds.sq.zero_()
    every = ds.linears + ([ds.lm] if ds.lm else [])
    if every:
        dp.dp_ghost_norms(every, ds.B, ds.T, ds.sq, ws=ds.ws, dev_status=ds.dev_status, stream=stream)
    if after_first_launch is not None:
        after_first_launch()
    if ds.vectors:
        dp.dp_vector_norms(ds.vectors, ds.B, ds.T, ds.sq, ws=ds.ws, stream=stream)
    dp.dp_embed_norms(ds.ids, ds.G_emb, ds.V, ds.sq, ws=ds.ws, dev_status=ds.dev_status, stream=stream)
    if ds.positions:
        dp.dp_embed_norms(ds.pos_ids, ds.G_emb, ds.T, ds.sq, ws=ds.ws, dev_status=ds.dev_status,
                          stream=stream)
    if ds.tied:
        dp.dp_tied_cross_term(ds.ids, ds.G_emb, ds.lm.A, ds.lm.G, ds.V, sq=ds.sq, cross=ds.cross,
                              d=ds.d_model, ws=ds.ws, dev_status=ds.dev_status, stream=stream)
    dp.dp_clip_factors(ds.sq, ds.C, clip=ds.clip, norms=ds.norms, stream=stream)


def _clip_vectors(ds: DeviceStep, beta: float, noise=None, stream=None, factors: bool = False) -> None:
    """Clipped sums of the bias / LayerNorm parameters (noise = (seed, step, scale) fuses Eq. 3)."""
    if not ds.vectors:
        return
    names = [f"vector{k}" for k in range(len(ds.vectors))]
    args = None
    if noise is not None:
        seed, step, scale = noise
        tid = tensor_ids(ds)
        args = (ds.sigma, scale, seed, [tid[n] for n in names], step)
    # factors=True: ds.clip already holds the clip factors of this step
    dp.dp_clip_accumulate_vectors(ds.vectors, ds.B, ds.T, None if factors else ds.sq, ds.C,
                                  [ds.outs[n] for n in names], beta=beta, noise=args, ws=ds.ws,
                                  stream=stream, clip=ds.clip if factors else None)


def clip_phase(ds: DeviceStep, stream=None, gemm_events=None) -> None:
    """Clipped sums of every parameter tensor from ds.sq."""
    kw = dict(ws=ds.ws, dev_status=ds.dev_status, stream=stream)
    layers = list(ds.linears)
    outs = [ds.outs[f"linear{k}"] for k in range(len(ds.linears))]
    if ds.lm is not None:
        layers.append(ds.lm)
        outs.append(ds.outs["wte"] if ds.tied else ds.outs["lm_head"])
    if layers:
        if gemm_events:
            gemm_events[0].record(torch.cuda.current_stream())
        dp.dp_clip_accumulate_grouped(layers, ds.B, ds.T, ds.sq, ds.C, outs, beta=0.0, **kw)
        if gemm_events:
            gemm_events[1].record(torch.cuda.current_stream())
    dp.dp_clip_accumulate_embed(ds.ids, ds.G_emb, ds.V, ds.sq, ds.C, ds.outs["wte"],
                                beta=1.0 if (ds.tied and ds.lm is not None) else 0.0, d=ds.d_model, **kw)
    if ds.positions:
        dp.dp_clip_accumulate_embed(ds.pos_ids, ds.G_emb, WPE_ROWS, ds.sq, ds.C, ds.outs["wpe"],
                                    beta=0.0, d=ds.d_model, **kw)
    _clip_vectors(ds, 0.0, stream=stream)


def clip_phase_bucketed(ds: DeviceStep, exchange, n_linear_buckets: int = 3) -> None:
    """Clipped sums produced bucket by bucket -- the LM head first (tied: together with the token
    scatter into the shared table), then the block linears in a few groups, then the remaining
    tables and vectors -- with `exchange.submit(names)` called right after each bucket's kernels
    were enqueued (a parallel.BucketedExchange: its collectives run on their own stream while the
    next bucket computes).  ds.clip must already hold the clip factors."""
    from . import parallel
    kw = dict(ws=ds.ws, dev_status=ds.dev_status)
    tied_head = ds.tied and ds.lm is not None

    def scatter_tokens(beta):
        dp.dp_clip_accumulate_embed(ds.ids, ds.G_emb, ds.V, None, ds.C, ds.outs["wte"], beta=beta,
                                    d=ds.d_model, clip=ds.clip, **kw)

    lin_names = [f"linear{k}" for k in range(len(ds.linears))]
    by_name = dict(zip(lin_names, ds.linears))
    head = None
    if ds.lm is not None:
        head = "wte" if ds.tied else "lm_head"
        by_name[head] = ds.lm
    last = ([] if tied_head else ["wte"]) + (["wpe"] if ds.positions else []) + \
           [f"vector{k}" for k in range(len(ds.vectors))]
    for bucket in parallel.bucket_order(lin_names, head, [], n_linear_buckets):
        layers = [by_name[n] for n in bucket]
        dp.dp_clip_accumulate_grouped(layers, ds.B, ds.T, None, ds.C, [ds.outs[n] for n in bucket],
                                      beta=0.0, clip=ds.clip, **kw)
        if tied_head and bucket == [head]:
            scatter_tokens(1.0)              # the shared table receives both contributions (Eq. 8)
        exchange.submit(bucket)
    if not tied_head:
        scatter_tokens(0.0)
    if ds.positions:
        dp.dp_clip_accumulate_embed(ds.pos_ids, ds.G_emb, WPE_ROWS, None, ds.C, ds.outs["wpe"],
                                    beta=0.0, d=ds.d_model, clip=ds.clip, **kw)
    _clip_vectors(ds, 0.0, factors=True)
    if last:
        exchange.submit(last)


def noise_phase(ds: DeviceStep, seed: int, step: int, scale: float = 1.0, stream=None) -> None:
    """One Gaussian draw per parameter tensor; tensor_id = position in the sorted key order."""
    for tid, name in enumerate(sorted(ds.outs)):
        dp.dp_add_noise(ds.outs[name], ds.sigma, ds.C, scale, seed, tid, step, stream=stream)


def tensor_ids(ds: DeviceStep) -> Dict[str, int]:
    return {name: tid for tid, name in enumerate(sorted(ds.outs))}


def clip_noise_phase(ds: DeviceStep, seed: int, step: int, scale: float = 1.0, stream=None) -> None:
    """Clipped sums with the noise fused in: same values as clip_phase + noise_phase, but the
    linear-layer noise is generated in the GEMM epilogue and the embedding table is filled with
    its noise instead of zeros (single-device use: no exchange between sum and noise)."""
    kw = dict(ws=ds.ws, dev_status=ds.dev_status, stream=stream)
    tid = tensor_ids(ds)
    layers = list(ds.linears)
    names = [f"linear{k}" for k in range(len(ds.linears))]
    if ds.lm is not None:
        layers.append(ds.lm)
        names.append("wte" if ds.tied else "lm_head")
    if layers:
        dp.dp_clip_accumulate_noise_grouped(layers, ds.B, ds.T, ds.sq, ds.C, [ds.outs[n] for n in names],
                                            ds.sigma, scale, seed, [tid[n] for n in names], step,
                                            beta=0.0, **kw)
    dp.dp_clip_accumulate_embed_noise(ds.ids, ds.G_emb, ds.V, ds.sq, ds.C, ds.outs["wte"], ds.sigma,
                                      scale, seed, tid["wte"], step,
                                      beta=1.0 if (ds.tied and ds.lm is not None) else 0.0,
                                      d=ds.d_model, **kw)
    if ds.positions:
        dp.dp_clip_accumulate_embed_noise(ds.pos_ids, ds.G_emb, WPE_ROWS, ds.sq, ds.C, ds.outs["wpe"],
                                          ds.sigma, scale, seed, tid["wpe"], step, beta=0.0,
                                          d=ds.d_model, **kw)
    _clip_vectors(ds, 0.0, noise=(seed, step, scale), stream=stream)


def prefill_embedding_noise(ds: DeviceStep, seed: int, step: int, scale: float = 1.0,
                            after: Optional[torch.cuda.Event] = None) -> torch.cuda.Event:
    """Start the noise fill of the embedding tables on a side stream.  The fill depends on no
    gradient, so it overlaps the (HBM-bound) norm phase; returns the event to wait for.
    after: event that orders the fill behind the previous users of the tables (default: all
    work enqueued so far on the current stream)."""
    if ds.side_stream is None:
        ds.side_stream = torch.cuda.Stream(device=ds.sq.device)
    main = torch.cuda.current_stream()
    tid = tensor_ids(ds)
    side = ds.side_stream
    if after is not None:
        side.wait_event(after)
    else:
        side.wait_stream(main)                   # previous step's readers of the tables are done
    names = ["wpe"] if ds.positions else []
    if not (ds.tied and ds.lm is not None):
        names.append("wte")                      # tied: the head GEMM writes the table first
    for name in names:
        dp.dp_fill_noise(ds.outs[name], ds.sigma, ds.C, scale, seed, tid[name], step, stream=side)
    ev = torch.cuda.Event()
    ev.record(side)
    return ev


def prefill_all_noise(ds: DeviceStep, seed: int, step: int) -> torch.cuda.Event:
    """Fill EVERY output tensor with its noise on the side stream (scale 1).  The fills are
    ALU-bound and depend on no gradient, the norm phase is HBM-bound: they share the SMs."""
    if ds.side_stream is None:
        ds.side_stream = torch.cuda.Stream(device=ds.sq.device)
    side = ds.side_stream
    side.wait_stream(torch.cuda.current_stream())
    for tid, name in enumerate(sorted(ds.outs)):
        dp.dp_fill_noise(ds.outs[name], ds.sigma, ds.C, 1.0, seed, tid, step, stream=side)
    ev = torch.cuda.Event()
    ev.record(side)
    return ev


def clip_onto_noise(ds: DeviceStep, filled: torch.cuda.Event) -> None:
    """Clipped sums accumulated (beta = 1) onto tensors that already hold their noise."""
    kw = dict(ws=ds.ws, dev_status=ds.dev_status)
    layers = list(ds.linears)
    names = [f"linear{k}" for k in range(len(ds.linears))]
    if ds.lm is not None:
        layers.append(ds.lm)
        names.append("wte" if ds.tied else "lm_head")
    torch.cuda.current_stream().wait_event(filled)
    if layers:
        dp.dp_clip_accumulate_grouped(layers, ds.B, ds.T, ds.sq, ds.C, [ds.outs[n] for n in names],
                                      beta=1.0, **kw)
    dp.dp_clip_accumulate_embed(ds.ids, ds.G_emb, ds.V, ds.sq, ds.C, ds.outs["wte"], beta=1.0,
                                d=ds.d_model, **kw)
    if ds.positions:
        dp.dp_clip_accumulate_embed(ds.pos_ids, ds.G_emb, WPE_ROWS, ds.sq, ds.C, ds.outs["wpe"],
                                    beta=1.0, d=ds.d_model, **kw)
    _clip_vectors(ds, 1.0)


def clip_after_prefill(ds: DeviceStep, seed: int, step: int, filled: torch.cuda.Event,
                       scale: float = 1.0, gemm_events=None) -> None:
    """Clipped sums when the embedding tables already hold their noise (see prefill).
    gemm_events: optional (start, stop) CUDA events recorded around the grouped GEMM call."""
    kw = dict(ws=ds.ws, dev_status=ds.dev_status)
    tid = tensor_ids(ds)
    layers = list(ds.linears)
    names = [f"linear{k}" for k in range(len(ds.linears))]
    if ds.lm is not None:
        layers.append(ds.lm)
        names.append("wte" if ds.tied else "lm_head")
    if layers:
        if gemm_events:
            gemm_events[0].record(torch.cuda.current_stream())
        # sq=None: ds.clip already holds the factors (overlapped_norms computed them)
        dp.dp_clip_accumulate_noise_grouped(layers, ds.B, ds.T, None, ds.C, [ds.outs[n] for n in names],
                                            ds.sigma, scale, seed, [tid[n] for n in names], step,
                                            beta=0.0, clip=ds.clip, **kw)
        if gemm_events:
            gemm_events[1].record(torch.cuda.current_stream())
    torch.cuda.current_stream().wait_event(filled)
    # beta = 1: rows are added onto the noise (untied) or onto head sum + noise (tied); the token
    # sorts were made beside the norm phase
    sb = ds.side
    dp.dp_clip_accumulate_embed_sorted(ds.ids, ds.G_emb, ds.V, None, ds.C, ds.outs["wte"], sb["perm"],
                                       sb["seg"], beta=1.0, d=ds.d_model, clip=ds.clip, **kw)
    if ds.positions:
        dp.dp_clip_accumulate_embed_sorted(ds.pos_ids, ds.G_emb, WPE_ROWS, None, ds.C, ds.outs["wpe"],
                                           sb["pos_perm"], sb["pos_seg"], beta=1.0, d=ds.d_model,
                                           clip=ds.clip, **kw)
    _clip_vectors(ds, 0.0, noise=(seed, step, scale), factors=True)


def _side_buffers(ds: DeviceStep) -> dict:
    """Buffers of the side stream (allocated once): it runs beside the main stream, so it needs its
    own workspace and its own norm accumulator; the token sorts it makes are kept for the scatter."""
    if ds.side is None:
        dev = ds.sq.device
        L = dp.load()
        rows = max(ds.V, WPE_ROWS if ds.positions else 0)
        need = max(int(L.dp_embed_norms_ws_bytes(ds.B, ds.T, ds.d_model)),
                   int(L.dp_embed_sort_ws_bytes(ds.B, ds.T, rows)), 256)
        ds.side = dict(
            ws=torch.empty(need, dtype=torch.uint8, device=dev),
            sq=torch.zeros(ds.B, dtype=torch.float32, device=dev),
            perm=torch.empty(ds.B * ds.T, dtype=torch.int32, device=dev),
            seg=torch.empty(ds.V + 1, dtype=torch.int32, device=dev),
            pos_perm=torch.empty(ds.B * ds.T, dtype=torch.int32, device=dev) if ds.positions else None,
            pos_seg=torch.empty(WPE_ROWS + 1, dtype=torch.int32, device=dev) if ds.positions else None)
    return ds.side


def overlapped_norms(ds: DeviceStep, seed: int, step: int) -> torch.cuda.Event:
    """Norm phase with everything that does not need the big norm kernel running BESIDE it on a
    side stream: the embedding norms (small kernels), the token sorts of the scatter (they need
    only the ids) and the embedding tables' noise fill (ALU-bound, depends on no gradient).  The
    side work is enqueued right AFTER the big kernel: measured on B200, work that is already
    resident keeps the norm kernel's CTAs out until it ends, while work that arrives second shares
    the SMs.  Returns the event after which the tables hold their noise and the sorts exist."""
    main = torch.cuda.current_stream()
    if ds.side_stream is None:
        ds.side_stream = torch.cuda.Stream(device=ds.sq.device)
    side, sb = ds.side_stream, _side_buffers(ds)
    start = torch.cuda.Event()
    start.record(main)
    ds.sq.zero_()
    every = ds.linears + ([ds.lm] if ds.lm else [])
    if every:
        dp.dp_ghost_norms(every, ds.B, ds.T, ds.sq, ws=ds.ws, dev_status=ds.dev_status)
    # ---- side stream
    side.wait_event(start)                       # previous step's readers of these buffers are done
    with torch.cuda.stream(side):
        sb["sq"].zero_()
    kw = dict(ws=sb["ws"], dev_status=ds.dev_status, stream=side)
    dp.dp_embed_norms(ds.ids, ds.G_emb, ds.V, sb["sq"], **kw)
    if ds.positions:
        dp.dp_embed_norms(ds.pos_ids, ds.G_emb, ds.T, sb["sq"], **kw)
    normed = torch.cuda.Event()
    normed.record(side)
    dp.dp_embed_sort(ds.ids, ds.V, sb["perm"], sb["seg"], **kw)
    if ds.positions:
        dp.dp_embed_sort(ds.pos_ids, WPE_ROWS, sb["pos_perm"], sb["pos_seg"], **kw)
    filled = prefill_embedding_noise(ds, seed, step, after=start)
    # ---- main stream again
    if ds.vectors:
        dp.dp_vector_norms(ds.vectors, ds.B, ds.T, ds.sq, ws=ds.ws)
    if ds.tied:
        dp.dp_tied_cross_term(ds.ids, ds.G_emb, ds.lm.A, ds.lm.G, ds.V, sq=ds.sq, cross=ds.cross,
                              d=ds.d_model, ws=ds.ws, dev_status=ds.dev_status)
    main.wait_event(normed)
    # join the two accumulators (one fixed order of additions: deterministic) and take Eq. 7
    dp.dp_clip_factors_sum(ds.sq, sb["sq"], ds.C, clip=ds.clip, norms=ds.norms)
    return filled


def dp_step(ds: DeviceStep, seed: int = 0, step: int = 0, noise: bool = True, fused: bool = True,
            overlap: bool = True, stream=None, events=None) -> None:
    """norms -> clipped sums -> noise.

    fused=True draws the linear-layer noise inside the clipped-sum GEMM; with overlap=True the
    embedding tables' noise is filled on a side stream while the norms run (scale 1 only).
    """
    if noise and fused and overlap and stream is None:
        # events (optional, default path only): five CUDA events recorded at step start, after the
        # norm phase, around the grouped GEMM call and at step end
        cur = torch.cuda.current_stream()
        if events: events[0].record(cur)
        filled = overlapped_norms(ds, seed, step)
        if events: events[1].record(cur)
        clip_after_prefill(ds, seed, step, filled, gemm_events=(events[2], events[3]) if events else None)
        if events: events[4].record(cur)
        return
    norms_phase(ds, stream)
    if noise and fused:
        clip_noise_phase(ds, seed, step, stream=stream)
        return
    clip_phase(ds, stream)
    if noise:
        noise_phase(ds, seed, step, stream=stream)


class StepGraph:
    """One whole step (norms -> clipped sums -> noise) captured once into a CUDA graph.

    The noise `step` word cannot be baked into the captured launches, so the kernels read a device
    counter (dp_noise_step_device) that the graph itself increments: replay k draws the stream of
    step `first_step + k`, exactly what `dp_step(ds, seed, step=first_step + k)` draws.  The graph
    holds the addresses of `ds`'s tensors: refill them in place between replays.
    """

    def __init__(self, ds: DeviceStep, seed: int = 0, first_step: int = 0, timing: bool = False):
        self.ds = ds
        # timing=True: external events inside the graph (step start, norms done, GEMM start, GEMM
        # end, step end), readable after a replay has completed
        self.events = ([torch.cuda.Event(enable_timing=True, external=True) for _ in range(5)]
                       if timing else None)
        dev = ds.sq.device
        self.counter = torch.full((1,), int(first_step), dtype=torch.int32, device=dev)
        # one eager step first: one-time kernel attribute setup must not happen during capture
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            dp_step(ds, seed=seed, step=first_step)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize(dev)
        self.graph = torch.cuda.CUDAGraph()
        dp.dp_noise_step_device(self.counter)
        try:
            n0 = dp.dp_kernel_launches()
            with torch.cuda.graph(self.graph):
                dp_step(ds, seed=seed, step=0, events=self.events)
                self.counter.add_(1)
            self.kernels_per_replay = dp.dp_kernel_launches() - n0    # this library's kernels
        finally:
            dp.dp_noise_step_device(None)        # eager calls made later take their step as given

    def replay(self) -> None:
        self.graph.replay()

    def phase_ms(self) -> dict:
        """Durations inside the LAST completed replay (timing=True; synchronize first)."""
        e = self.events
        return {"norms": e[0].elapsed_time(e[1]), "clip_accumulate": e[1].elapsed_time(e[4]),
                "gemm": e[2].elapsed_time(e[3]), "step": e[0].elapsed_time(e[4])}
