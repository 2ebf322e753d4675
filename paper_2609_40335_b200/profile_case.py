"""Small single-kernel cases for profilers (each runs one entry point a few times on cuda:0).

    python -m paper_2609_40335_b200.profile_case gemm|ghost|ghost512|noise|embed|embed_small|cross|vectors [reps]

Sizes are chosen so that inputs exceed the 126 MB L2 but stay well under a few GB, which keeps
a multi-pass `ncu` capture short.
"""
from __future__ import annotations

import sys

import torch

from . import binding as dp


def _randn_bf16(*shape, std=1.0):
    return (torch.randn(*shape, device="cuda") * std).to(torch.bfloat16)


def case_gemm(reps, sq_value=4.0):
    B, T = 32, 128
    # 148 x 3 output tiles of 128 x 256: exactly three full waves on 148 SMs
    layers = [dp.Linear(_randn_bf16(B, T, 768), _randn_bf16(B, T, 148 * 128, std=1e-2))]
    outs = [torch.empty(l.G.shape[-1], l.A.shape[-1], device="cuda") for l in layers]
    sq = torch.full((B,), sq_value, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dp.dp_clip_accumulate_grouped(layers, B, T, sq, 1.0, outs)
    e0.record()
    for _ in range(reps):
        dp.dp_clip_accumulate_grouped(layers, B, T, sq, 1.0, outs)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    flops = sum(2 * B * T * l.A.shape[-1] * l.G.shape[-1] for l in layers)
    print(f"gemm: {ms:.4f} ms per call, {flops / ms / 1e9:.1f} TFLOP/s (clip {'on' if sq_value > 1 else 'off'})")


def case_gemm_unclipped(reps):
    case_gemm(reps, sq_value=1e-12)


def case_ghost(reps):
    B, T = 32, 128
    layers = [dp.Linear(_randn_bf16(B, T, 768), _randn_bf16(B, T, 3072, std=1e-2)) for _ in range(6)]
    layers.append(dp.Linear(_randn_bf16(B, T, 768), _randn_bf16(B, T, 16384, std=1e-2)))
    sq = torch.zeros(B, device="cuda")
    for _ in range(reps):
        dp.dp_ghost_norms(layers, B, T, sq)


def case_ghost_long(reps):
    """Tensor-bound regime of the ghost norm: T = 512 (10 tile pairs per example and layer)."""
    B, T = 64, 512
    layers = [dp.Linear(_randn_bf16(B, T, 1024), _randn_bf16(B, T, 4096, std=1e-2)) for _ in range(2)]
    sq = torch.zeros(B, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dp.dp_ghost_norms(layers, B, T, sq)
    e0.record()
    for _ in range(reps):
        dp.dp_ghost_norms(layers, B, T, sq)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    tiles = 10 * B * len(layers)                       # 128 x 128 tile pairs
    flops = tiles * 2 * 128 * 128 * (1024 + 4096)
    nbytes = B * len(layers) * 2 * T * (1024 + 4096)
    print(f"ghost T=512: {ms:.4f} ms per call, {flops / ms / 1e9:.1f} TFLOP/s issued, "
          f"{nbytes / ms / 1e6:.0f} GB/s algorithmic")


def case_overlap(reps):
    """Does the ALU-bound noise fill share the SMs with the HBM-bound norm kernel?"""
    B, T = 32, 128
    layers = [dp.Linear(_randn_bf16(B, T, 768), _randn_bf16(B, T, 3072, std=1e-2)) for _ in range(18)]
    sq = torch.zeros(B, device="cuda")
    x = torch.empty(50257 * 768, device="cuda")
    side = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    ws = torch.empty(dp.dp_ghost_norms_ws_bytes(layers, B, T), dtype=torch.uint8, device="cuda")

    def run(mode):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(main)
        for k in range(reps):
            if mode in ("fill", "fill_first"):
                side.wait_stream(main)
                dp.dp_fill_noise(x, 0.8, 1.0, 1.0, 1, 0, k, stream=side)
            if mode != "fill":
                dp.dp_ghost_norms(layers, B, T, sq, ws=ws)
            if mode == "ghost_first":
                side.wait_stream(main) if False else None
                dp.dp_fill_noise(x, 0.8, 1.0, 1.0, 1, 0, k, stream=side)
            main.wait_stream(side)
        e1.record(main)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    for mode in ("ghost", "fill", "fill_first", "ghost_first"):
        run(mode)
        print(f"overlap[{mode}]: {run(mode):.4f} ms per iteration")


def case_noise(reps):
    x = torch.zeros(50257 * 768, device="cuda")
    for k in range(reps):
        dp.dp_add_noise(x, 0.8, 1.0, 1.0, 1234, 0, k)


def case_embed(reps, B=256, T=512, d=1024):
    V = 50257
    w = torch.arange(1, V + 1, device="cuda", dtype=torch.float64) ** -1.1
    ids = torch.multinomial(w / w.sum(), B * T, replacement=True).to(torch.int32).view(B, T)
    G = _randn_bf16(B, T, d, std=1e-2)
    sq = torch.zeros(B, device="cuda")
    out = torch.empty(V, d, device="cuda")
    for _ in range(reps):
        dp.dp_embed_norms(ids, G, V, sq)
        dp.dp_clip_accumulate_embed(ids, G, V, sq, 1.0, out)


def case_embed_small(reps):
    case_embed(reps, B=32, T=128, d=768)


def case_cross(reps):
    B, T, d, V = 32, 128, 768, 50257
    ids = torch.randint(0, V, (B, T), device="cuda", dtype=torch.int32)
    G_emb, A_lm = _randn_bf16(B, T, d, std=1e-2), _randn_bf16(B, T, d)
    G_lm = _randn_bf16(B, T, 50264, std=1e-2)
    sq = torch.zeros(B, device="cuda")
    for _ in range(reps):
        dp.dp_tied_cross_term(ids, G_emb, A_lm, G_lm, V, sq=sq, d=d)


def case_vectors(reps):
    """Bias and LayerNorm parameters of 6 GPT-2 blocks at B=32, T=128 (norms, then clipped sums)."""
    B, T = 32, 128
    vec = []
    for _ in range(6):
        for p_, with_x in [(768, True), (768, False), (2304, False), (768, False), (768, True), (768, False),
                           (3072, False), (768, False)]:
            G = _randn_bf16(B, T, p_, std=1e-2)
            vec.append(dp.Vector(G, _randn_bf16(B, T, p_) if with_x else None, p=p_))
    sq = torch.zeros(B, device="cuda")
    outs = [torch.empty(v.p, device="cuda") for v in vec]
    for _ in range(reps):
        dp.dp_vector_norms(vec, B, T, sq)
        dp.dp_clip_accumulate_vectors(vec, B, T, sq, 1.0, outs)


def main():
    which = sys.argv[1] if len(sys.argv) > 1 else "gemm"
    reps = int(sys.argv[2]) if len(sys.argv) > 2 else 3
    torch.manual_seed(0)
    {"gemm": case_gemm, "gemm1": case_gemm_unclipped, "ghost512": case_ghost_long, "overlap": case_overlap, "ghost": case_ghost, "noise": case_noise, "embed": case_embed, "embed_small": case_embed_small,
     "cross": case_cross, "vectors": case_vectors}[which](reps)
    torch.cuda.synchronize()
    print("done", which, reps)


if __name__ == "__main__":
    main()
