"""Seeded synthetic inputs for the DP-SGD hot path (numpy only, host memory).

This module serves both the CUDA path and the float64 test oracle, so it holds
none of the method's arithmetic: it only draws random tensors with the shapes
and value distributions of GPT-2-style fine-tuning (layer sizes, vocabulary,
Zipf token frequencies) and rounds them to the storage type.

bf16 tensors are carried as uint16 bit patterns (numpy has no bf16); the same
bits go to the device and, widened exactly, to the oracle.
"""
from __future__ import annotations

import dataclasses
import hashlib
from typing import List, Optional, Tuple

import numpy as np

GPT2_VOCAB = 50257


# ----------------------------------------------------------------------- bf16 bits
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclasses.dataclass
class HostTensor:
    """A host tensor in its storage type.

    data: fp32 array, or uint16 bf16 bit patterns; shape (..., ld) with the
    logical width `cols` <= ld (columns cols..ld-1 are padding the method must
    never read; they are filled with NaN to prove it).
    """
    data: np.ndarray
    dtype: str            # "f32" | "bf16"
    cols: int

    @property
    def ld(self) -> int:
        return self.data.shape[-1]

    def widened(self) -> np.ndarray:
        """Logical values as float64 (padding dropped)."""
        v = self.data if self.dtype == "f32" else bf16_bits_to_f32(self.data)
        return v[..., : self.cols].astype(np.float64)

    def widened_rows(self, sl) -> np.ndarray:
        """Logical float64 values of a slice along the first axis (saves memory)."""
        d = self.data[sl]
        v = d if self.dtype == "f32" else bf16_bits_to_f32(d)
        return v[..., : self.cols].astype(np.float64)


def _seed_for(base_seed: int, *tag) -> int:
    h = hashlib.sha256(repr((int(base_seed),) + tuple(tag)).encode()).digest()
    return int.from_bytes(h[:8], "little")


_CHUNK_ELEMS = 1 << 24


def _normal_jobs(shape, std, dtype, seed, ld=None):
    """The tensor (allocated, not yet filled) and the jobs that fill it.

    A tensor is drawn in slabs along its first axis, at most 2^24 elements each and every slab from
    its own generator (seeded by the tensor's seed and the slab number), so that the slabs can be
    drawn in parallel and the values depend on the shape and the seed only -- not on how many
    threads draw them.  A tensor of one slab uses the tensor's seed itself.
    """
    shape = tuple(int(v) for v in shape)
    cols = shape[-1]
    ld = cols if ld is None else int(ld)
    out = np.empty(shape[:-1] + (ld,), dtype=np.uint16 if dtype == "bf16" else np.float32)
    per_row = int(np.prod(shape[1:], dtype=np.int64))
    rows = max(1, _CHUNK_ELEMS // max(per_row, 1))
    n_slabs = (shape[0] + rows - 1) // rows

    def fill(k):
        r0, r1 = k * rows, min(shape[0], (k + 1) * rows)
        rng = np.random.Generator(np.random.PCG64(seed if n_slabs == 1 else _seed_for(seed, "slab", k)))
        x = rng.standard_normal(size=(r1 - r0,) + shape[1:], dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        if ld != cols:
            full = np.full((r1 - r0,) + shape[1:-1] + (ld,), np.nan, dtype=np.float32)
            full[..., :cols] = x
            x = full
        out[r0:r1] = f32_to_bf16_bits(x) if dtype == "bf16" else x

    return HostTensor(out, dtype, cols), [(fill, k) for k in range(n_slabs)]


def _run_jobs(jobs) -> None:
    """Run fill jobs on a thread pool (numpy's generators and ufuncs release the GIL)."""
    import concurrent.futures as cf
    import os
    workers = max(1, min(16, len(os.sched_getaffinity(0)), len(jobs)))
    if workers == 1:
        for fn, k in jobs:
            fn(k)
        return
    with cf.ThreadPoolExecutor(max_workers=workers) as ex:
        list(ex.map(lambda j: j[0](j[1]), jobs))


def _normal(shape, std, dtype, seed, ld=None) -> HostTensor:
    t, jobs = _normal_jobs(shape, std, dtype, seed, ld)
    _run_jobs(jobs)
    return t


def zipf_ids(B: int, T: int, V: int, s: float, seed: int) -> np.ndarray:
    """Token ids with P(id = k-1) proportional to k^-s on k = 1..V (bounded Zipf)."""
    w = np.arange(1, V + 1, dtype=np.float64) ** (-float(s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    rng = np.random.Generator(np.random.PCG64(seed))
    u = rng.random(size=(B, T))
    ids = np.searchsorted(cdf, u, side="right")
    return np.minimum(ids, V - 1).astype(np.int32)


def uniform_ids(B: int, T: int, V: int, seed: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, V, size=(B, T), dtype=np.int32)


@dataclasses.dataclass
class LinearIO:
    name: str
    d: int
    p: int
    A: HostTensor         # (B, T, d)
    G: HostTensor         # (B, T, p)


@dataclasses.dataclass
class VectorIO:
    """A bias or LayerNorm parameter: gradient G (B, T, p) at its output and, for a LayerNorm
    gain, the normalised input X (B, T, p); X is None for biases and LayerNorm shifts."""
    name: str
    p: int
    G: HostTensor
    X: Optional[HostTensor]


@dataclasses.dataclass
class Workload:
    name: str
    dtype: str
    B: int
    T: int
    V: int
    C: float
    sigma: float
    seed: int
    linears: List[LinearIO]
    ids: np.ndarray                       # (B, T) int32
    G_emb: HostTensor                     # (B, T, d_model)
    lm: Optional[LinearIO]                # LM head (A_lm, G_lm) or None
    tied: bool
    positions: bool
    vectors: List[VectorIO] = dataclasses.field(default_factory=list)

    @property
    def d_model(self) -> int:
        return self.G_emb.cols


def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def make_workload(name: str, *, B: int, T: int, dtype: str,
                  block_shapes: List[Tuple[int, int]], n_blocks: int, d_model: int,
                  V: int, lm_head: bool, tied: bool = False, positions: bool = False,
                  C: float = 1.0, sigma: float = 1.0, id_dist: str = "zipf",
                  a_std: float = 1.0, g_std: float = 1e-2, seed: int = 0,
                  shared_block_inputs: bool = False, full_model: bool = False) -> Workload:
    """Draw one workload.

    block_shapes: the (d, p) of the linear layers inside one transformer block.
    g_std: standard deviation of output gradients ("N(0, 1e-4)" is read as a
    variance, like the paper's N(0, sigma^2 C^2 I)).  shared_block_inputs: draw
    one tensor set per distinct layer shape and reuse it in every block (used
    only where the full set would not fit in host memory).  full_model: also emit the
    biases of the block linears and the LayerNorm gains / shifts of a GPT-2 block (ln_1, ln_2,
    final ln_f), so that the parameter blocks cover the whole model.
    """
    jobs = []

    def _normal(shape, std, dtype, seed, ld=None):        # deferred: all tensors are drawn together
        t, j = _normal_jobs(shape, std, dtype, seed, ld)
        jobs.extend(j)
        return t

    linears: List[LinearIO] = []
    cache = {}
    for blk in range(n_blocks):
        for li, (d, p) in enumerate(block_shapes):
            key = (li,) if shared_block_inputs else (blk, li)
            if key not in cache:
                A = _normal((B, T, d), a_std, dtype, _seed_for(seed, name, "A", key))
                G = _normal((B, T, p), g_std, dtype, _seed_for(seed, name, "G", key))
                cache[key] = (A, G)
            A, G = cache[key]
            linears.append(LinearIO(f"h{blk}.l{li}_{d}x{p}", d, p, A, G))
    if id_dist == "zipf":
        ids = zipf_ids(B, T, V, 1.1, _seed_for(seed, name, "ids"))
    elif id_dist == "uniform":
        ids = uniform_ids(B, T, V, _seed_for(seed, name, "ids"))
    else:
        raise ValueError(id_dist)
    G_emb = _normal((B, T, d_model), g_std, dtype, _seed_for(seed, name, "G_emb"))
    lm = None
    if lm_head:
        ld = round_up(V, 8) if dtype == "bf16" else V
        A_lm = _normal((B, T, d_model), a_std, dtype, _seed_for(seed, name, "A_lm"))
        G_lm = _normal((B, T, V), g_std, dtype, _seed_for(seed, name, "G_lm"), ld=ld)
        lm = LinearIO(f"lm_head_{d_model}x{V}", d_model, V, A_lm, G_lm)
    vectors: List[VectorIO] = []
    if full_model:
        per_block = len(block_shapes)

        ln_cache = {}

        def layer_norm(tag):
            if tag in ln_cache:
                return ln_cache[tag]
            G = _normal((B, T, d_model), g_std, dtype, _seed_for(seed, name, "G_ln", tag))
            X = _normal((B, T, d_model), 1.0, dtype, _seed_for(seed, name, "X_ln", tag))
            ln_cache[tag] = [VectorIO(f"{tag}.gamma", d_model, G, X),
                             VectorIO(f"{tag}.beta", d_model, G, None)]
            return ln_cache[tag]

        for blk in range(n_blocks):
            key = 0 if shared_block_inputs else blk
            vectors += layer_norm(f"h{key}.ln_1")
            if per_block == 4:
                vectors += layer_norm(f"h{key}.ln_2")
            for li in range(per_block):                    # the bias sees the linear layer's G
                l = linears[blk * per_block + li]
                vectors.append(VectorIO(f"{l.name}.bias", l.p, l.G, None))
        vectors += layer_norm("ln_f")
    _run_jobs(jobs)
    return Workload(name, dtype, B, T, V, float(C), float(sigma), seed, linears, ids, G_emb,
                    lm, tied, positions, vectors)


def gpt2_block_shapes(d_model: int) -> List[Tuple[int, int]]:
    """qkv, attention projection, MLP up, MLP down of one GPT-2 block."""
    return [(d_model, 3 * d_model), (d_model, d_model), (d_model, 4 * d_model),
            (4 * d_model, d_model)]


def named_workload(name: str, seed: int = 0, **over) -> Workload:
    """The five benchmark configurations (and scaled-down variants via overrides).

    cfg1: one fp32 linear 64->64 plus a V=1000 embedding, B=4, T=16, N(0,1) values.
    cfg2: DistilGPT2 shape, 6 blocks, d=768, B=32, T=128, untied head, sigma=0.8.
    cfg3: GPT-2-small shape, 12 blocks, B=64, T=256, untied head, position table.
    cfg4: GPT-2-small shape, 12 blocks, B=32, T=128, tied head.
    cfg5: GPT-2-medium shape, 24 blocks, d=1024; pass B= and T=.
    """
    if name == "cfg1":
        kw = dict(B=4, T=16, dtype="f32", block_shapes=[(64, 64)], n_blocks=1, d_model=64,
                  V=1000, lm_head=False, C=1.0, sigma=1.0, id_dist="uniform",
                  a_std=1.0, g_std=1.0)
    elif name == "cfg2":
        kw = dict(B=32, T=128, dtype="bf16", block_shapes=gpt2_block_shapes(768), n_blocks=6,
                  d_model=768, V=GPT2_VOCAB, lm_head=True, C=1.0, sigma=0.8)
    elif name == "cfg3":
        kw = dict(B=64, T=256, dtype="bf16", block_shapes=gpt2_block_shapes(768), n_blocks=12,
                  d_model=768, V=GPT2_VOCAB, lm_head=True, positions=True, C=1.0, sigma=0.8)
    elif name == "cfg4":
        kw = dict(B=32, T=128, dtype="bf16", block_shapes=gpt2_block_shapes(768), n_blocks=12,
                  d_model=768, V=GPT2_VOCAB, lm_head=True, tied=True, C=1.0, sigma=0.8)
    elif name == "cfg5":
        kw = dict(B=16, T=128, dtype="bf16", block_shapes=gpt2_block_shapes(1024), n_blocks=24,
                  d_model=1024, V=GPT2_VOCAB, lm_head=True, C=1.0, sigma=1.0,
                  shared_block_inputs=True)
    else:
        raise ValueError(f"unknown workload {name!r}")
    kw.update(over)
    return make_workload(name, seed=seed, **kw)
