"""Seeded random-shape parity: the linear-layer norms and clipped sums (single and grouped calls),
the embedding norm / sort / scatter, the tied cross term, the noise stream (stand-alone slices and
fused into the clipped sums) and the bias / LayerNorm parameters on shapes drawn at random -- ragged T,
d, p and V, padded leading dimensions (the padding holds NaN), every norm mode, both input types --
each compared with the oracle.  The fixed cases of test_gpu_parity.py pin the shapes of the
workloads; this file looks for the shape nobody thought of."""
import numpy as np
import pytest
import torch

from oracle import dp_oracle as O
from oracle import noise_oracle as NO
from paper_2609_40335_b200 import binding as dp
from paper_2609_40335_b200 import pipeline as P
from paper_2609_40335_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _dev():
    return torch.device("cuda:0")


def rel(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return np.abs(a - b) / np.maximum(np.abs(b), 1e-300)


def frob_rel(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def pick(rng, choices):
    return choices[int(rng.integers(len(choices)))]


def rand_dim(rng):
    kind = int(rng.integers(5))
    if kind == 0:
        v = int(rng.integers(1, 64))
    elif kind == 1:
        v = int(rng.integers(64, 300))
    elif kind == 2:
        v = pick(rng, [64, 128, 256, 512, 768, 1024])
    elif kind == 3:
        v = int(rng.integers(300, 1400))
    else:
        v = pick(rng, [63, 65, 127, 129, 255, 257, 1000, 2304])
    return v


def linear_case(rng, k):
    dtype = pick(rng, ["bf16", "bf16", "bf16", "f32"])
    B = int(rng.integers(1, 7))
    T = pick(rng, [1, 2, 7, 16, 31, 32, 33, 64, 100, 127, 128, 129, 130, 200, 255, 256, 257, 300, 384, 512, 513, 600])
    d, p = rand_dim(rng), rand_dim(rng)
    # keep the oracle affordable
    while B * T * d * p > 6e8:
        B = max(1, B // 2)
        if B == 1:
            d = max(8, d // 2)
    pad_g = int(rng.integers(3)) == 0
    ldg = None
    if dtype == "bf16":
        # tensor-core path wants ld % 8 == 0: the generator pads to it when cols are odd
        ldg = W.round_up(p, 8) + (8 * int(rng.integers(1, 4)) if pad_g else 0)
        if ldg == p:
            ldg = None
    elif pad_g:
        ldg = p + int(rng.integers(1, 9))
    seed = int(rng.integers(1 << 40))
    r2 = np.random.default_rng(seed)
    lda = None
    if dtype == "bf16" and d % 8:
        lda = W.round_up(d, 8)
    A = W._normal((B, T, d), 1.0, dtype, int(r2.integers(1 << 60)), ld=lda)
    G = W._normal((B, T, p), 1e-2, dtype, int(r2.integers(1 << 60)), ld=ldg)
    mode = pick(rng, [dp.DP_NORM_AUTO, dp.DP_NORM_GHOST, dp.DP_NORM_DIRECT])
    desc = f"#{k} {dtype} B{B} T{T} d{d} p{p} lda{lda} ldg{ldg} mode{mode}"
    lin = dp.Linear(P.to_device(A), P.to_device(G), d=d, p=p, mode=mode)
    sq = torch.zeros(B, device=_dev())
    st = torch.zeros(1, dtype=torch.int32, device=_dev())
    dp.dp_ghost_norms([lin], B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    bad = []
    if int(st.item()) != 0:
        bad.append(f"status {int(st.item())}")
    want = O.linear_sq_norms(A.widened(), G.widened())
    got = sq.cpu().numpy()
    tol = 2e-3 if dtype == "bf16" else 1e-4
    e = rel(got, want).max()
    if not np.isfinite(got).all() or e > tol:
        bad.append(f"norm err {e:.3e}")
    # clipped sum
    Cc = float(np.median(np.sqrt(want))) if B > 1 else float(np.sqrt(want[0]) * pick(rng, [0.5, 2.0]))
    beta = pick(rng, [0.0, 1.0])
    sqd = torch.from_numpy(want.astype(np.float32)).to(_dev())
    ldo_pad = pick(rng, [0, 0, 4])
    out0 = torch.randn(p, d + ldo_pad, device=_dev())
    out = out0.clone()
    clip = torch.zeros(B, device=_dev())
    st.zero_()
    outv = out[:, :d] if ldo_pad else out
    try:
        dp.dp_clip_accumulate(P.to_device(A), P.to_device(G), sqd, Cc, outv, beta=beta, d=d, p=p, clip=clip, dev_status=st)
    except Exception as ex:  # noqa: BLE001
        bad.append(f"clip_accumulate raised {ex}")
        return desc, bad
    torch.cuda.synchronize()
    if int(st.item()) != 0:
        bad.append(f"status2 {int(st.item())}")
    _, R = O.clip_factors(sqd.cpu().numpy().astype(np.float64), Cc)
    if rel(clip.cpu().numpy(), R).max() > 1e-6:
        bad.append("clip factors")
    wsum = O.clipped_sum_linear(A.widened(), G.widened(), R) + beta * out0[:, :d].cpu().numpy().astype(np.float64)
    fe = frob_rel(out[:, :d].cpu().numpy(), wsum)
    if fe > (5e-3 if dtype == "bf16" else 1e-4):
        bad.append(f"sum err {fe:.3e}")
    if ldo_pad and not torch.equal(out[:, d:], out0[:, d:]):
        bad.append("padding columns of out were written")
    return desc, bad


def rand_ids(rng, B, T, V):
    kind = int(rng.integers(4))
    seed = int(rng.integers(1 << 40))
    if kind == 0:
        ids = W.zipf_ids(B, T, V, 1.1, seed)
    elif kind == 1:
        ids = W.uniform_ids(B, T, V, seed)
    elif kind == 2:
        ids = W.uniform_ids(B, T, min(V, 3), seed)         # heavy duplication
    else:
        ids = W.zipf_ids(B, T, V, 2.0, seed)
    if B > 1 and int(rng.integers(3)) == 0:
        ids[0, :] = ids[0, 0]
    return ids


def embed_case(rng, k):
    dtype = pick(rng, ["bf16", "f32"])
    B = int(rng.integers(1, 6))
    T = pick(rng, [1, 2, 5, 16, 31, 32, 33, 64, 100, 128, 129, 255, 256, 300, 512, 700, 1024])
    d = pick(rng, [1, 3, 8, 10, 64, 96, 100, 132, 255, 256, 257, 300, 512, 768, 1000, 1024])
    V = pick(rng, [1, 2, 5, 7, 33, 300, 1000, 1024, 1025, 4099, 50257])
    ids = rand_ids(rng, B, T, V)
    ldd = W.round_up(d, 8) if (dtype == "bf16" and d % 8) else None
    gstd = 1.0 if dtype == "f32" else 1e-2
    G = W._normal((B, T, d), gstd, dtype, int(rng.integers(1 << 60)), ld=ldd)
    desc = f"#{k} embed {dtype} B{B} T{T} d{d} V{V}"
    bad = []
    sq = torch.zeros(B, device=_dev())
    fo = torch.full((B, T), -1, dtype=torch.int32, device=_dev())
    st = torch.zeros(1, dtype=torch.int32, device=_dev())
    idsd = torch.from_numpy(ids).to(_dev())
    dp.dp_embed_norms(idsd, P.to_device(G), V, sq, d=d, first_occ=fo, dev_status=st)
    torch.cuda.synchronize()
    if int(st.item()):
        bad.append(f"status {int(st.item())}")
    if not np.array_equal(fo.cpu().numpy(), O.first_occurrence(ids)):
        bad.append("first occurrence")
    want = O.embed_sq_norms(ids, G.widened(), V)
    tol = 1e-4 if dtype == "f32" else 2e-3
    e = rel(sq.cpu().numpy(), want).max()
    if e > tol:
        bad.append(f"embed norm err {e:.3e}")
    # clipped scatter
    Cc = float(np.median(np.sqrt(want)))
    beta = pick(rng, [0.0, 1.0])
    sqd = torch.from_numpy(want.astype(np.float32)).to(_dev())
    out0 = torch.randn(V, d, device=_dev())
    out = out0.clone()
    perm = torch.full((B * T,), -1, dtype=torch.int32, device=_dev())
    seg = torch.full((V + 1,), -1, dtype=torch.int32, device=_dev())
    st.zero_()
    dp.dp_clip_accumulate_embed(idsd, P.to_device(G), V, sqd, Cc, out, beta=beta, perm=perm, seg=seg, d=d,
                                dev_status=st)
    torch.cuda.synchronize()
    if int(st.item()):
        bad.append(f"status2 {int(st.item())}")
    wp, ws_ = O.stable_token_sort(ids, V)
    if not np.array_equal(perm.cpu().numpy(), wp) or not np.array_equal(seg.cpu().numpy(), ws_):
        bad.append("sort")
    _, R = O.clip_factors(sqd.cpu().numpy().astype(np.float64), Cc)
    wsum = O.clipped_sum_embed(ids, G.widened(), R, V) + beta * out0.cpu().numpy().astype(np.float64)
    fe = frob_rel(out.cpu().numpy(), wsum)
    if fe > 1e-5:
        bad.append(f"scatter err {fe:.3e}")
    return desc, bad


def cross_case(rng, k):
    dtype = pick(rng, ["bf16", "f32"])
    B = int(rng.integers(1, 4))
    T = pick(rng, [1, 5, 16, 33, 64, 70, 128, 129, 200, 256, 300, 512])
    d = pick(rng, [8, 64, 100, 136, 256, 300, 768])
    V = pick(rng, [2, 33, 300, 1000, 4099, 50257])
    while B * T * V > 4e7:
        if B > 1:
            B -= 1
        else:
            T = max(1, T // 2)
    ids = rand_ids(rng, B, T, V)
    g_std = 1.0 if dtype == "f32" else 1e-2
    ldd = W.round_up(d, 8) if (dtype == "bf16" and d % 8) else None
    G_emb = W._normal((B, T, d), g_std, dtype, int(rng.integers(1 << 60)), ld=ldd)
    A_lm = W._normal((B, T, d), 1.0, dtype, int(rng.integers(1 << 60)), ld=ldd)
    ld = W.round_up(V, 8) if dtype == "bf16" else V
    G_lm = W._normal((B, T, V), g_std, dtype, int(rng.integers(1 << 60)), ld=ld if ld != V else None)
    desc = f"#{k} cross {dtype} B{B} T{T} d{d} V{V}"
    bad = []
    ref = O.tied_sq_norms(ids, G_emb.widened(), A_lm.widened(), G_lm.widened(), V)
    sq = torch.zeros(B, device=_dev())
    cross = torch.zeros(B, device=_dev())
    st = torch.zeros(1, dtype=torch.int32, device=_dev())
    dp.dp_tied_cross_term(torch.from_numpy(ids).to(_dev()), P.to_device(G_emb), P.to_device(A_lm),
                          P.to_device(G_lm), V, sq=sq, cross=cross, d=d, dev_status=st)
    torch.cuda.synchronize()
    if int(st.item()):
        bad.append(f"status {int(st.item())}")
    scale = np.sqrt(ref["in"] * ref["out"])
    tol = 1e-4 if dtype == "f32" else 2e-3
    e = (np.abs(cross.cpu().numpy() - ref["cross"]) / scale).max()
    if not e < tol:
        bad.append(f"cross err {e:.3e}")
    return desc, bad


def grouped_case(rng, k):
    """several bf16 layers of mixed shapes and modes in one call, then the grouped clipped sums"""
    B = int(rng.integers(1, 5))
    T = pick(rng, [16, 64, 100, 128, 129, 200, 256, 300, 512])
    n = int(rng.integers(2, 7))
    lays, hosts = [], []
    for _ in range(n):
        d, p = rand_dim(rng), rand_dim(rng)
        while B * T * d * p > 2e8:
            d = max(8, d // 2)
        lda = W.round_up(d, 8) if d % 8 else None
        ldg = W.round_up(p, 8) if p % 8 else None
        A = W._normal((B, T, d), 1.0, "bf16", int(rng.integers(1 << 60)), ld=lda)
        G = W._normal((B, T, p), 1e-2, "bf16", int(rng.integers(1 << 60)), ld=ldg)
        mode = pick(rng, [dp.DP_NORM_AUTO, dp.DP_NORM_GHOST, dp.DP_NORM_DIRECT])
        lays.append(dp.Linear(P.to_device(A), P.to_device(G), d=d, p=p, mode=mode))
        hosts.append((A, G, d, p))
    desc = f"#{k} grouped B{B} T{T} " + " ".join(f"{d}x{p}" for _, _, d, p in hosts)
    bad = []
    sq = torch.zeros(B, device=_dev())
    st = torch.zeros(1, dtype=torch.int32, device=_dev())
    dp.dp_ghost_norms(lays, B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    if int(st.item()):
        bad.append(f"status {int(st.item())}")
    want = sum(O.linear_sq_norms(A.widened(), G.widened()) for A, G, _, _ in hosts)
    e = rel(sq.cpu().numpy(), want).max()
    if not e < 2e-3:
        bad.append(f"norm err {e:.3e}")
    Cc = float(np.median(np.sqrt(want))) * pick(rng, [0.5, 1.0, 1.0, 100.0])
    sqd = torch.from_numpy(want.astype(np.float32)).to(_dev())
    beta = pick(rng, [0.0, 1.0])
    outs0 = [torch.randn(p, d, device=_dev()) for _, _, d, p in hosts]
    outs = [o.clone() for o in outs0]
    st.zero_()
    dp.dp_clip_accumulate_grouped(lays, B, T, sqd, Cc, outs, beta=beta, dev_status=st)
    torch.cuda.synchronize()
    if int(st.item()):
        bad.append(f"status2 {int(st.item())}")
    _, R = O.clip_factors(sqd.cpu().numpy().astype(np.float64), Cc)
    for (A, G, d, p), o, o0 in zip(hosts, outs, outs0):
        wsum = O.clipped_sum_linear(A.widened(), G.widened(), R) + beta * o0.cpu().numpy().astype(np.float64)
        fe = frob_rel(o.cpu().numpy(), wsum)
        if not fe < 5e-3:
            bad.append(f"sum err {d}x{p} {fe:.3e}")
    return desc, bad

def noise_case(rng, k):
    """stand-alone noise on a slice that starts anywhere on a counter boundary (the counter's high
    word included), with random keys; a buffer that is not 16-byte aligned is refused"""
    n = pick(rng, [1, 2, 3, 4, 5, 7, 8, 31, 100, 1023, 4096, 10007, 65537, 300001])
    first = 4 * int(rng.integers(0, 1 << 20)) * pick(rng, [0, 1, 1, 4097])
    seed = int(rng.integers(0, 1 << 63)) * 2 + int(rng.integers(2))
    tid, step = int(rng.integers(0, 1 << 32)), int(rng.integers(0, 1 << 31))
    sigma, C_, scale = float(rng.uniform(0.1, 2.0)), float(rng.uniform(0.1, 3.0)), pick(rng, [1.0, 0.5, 1.0 / 64])
    off = pick(rng, [0, 0, 4, 1, 2, 3])
    buf = torch.randn(n + 8, device=_dev())
    part = buf[off:off + n]
    base = part.clone()
    desc = f"#{k} noise n{n} first{first} off{off} tid{tid} step{step}"
    bad = []
    if off % 4:
        try:
            dp.dp_add_noise_slice(part, first, sigma, C_, scale, seed, tid, step)
            bad.append("misaligned buffer accepted")
        except dp.DpGhostError as e:
            if e.status != 3:
                bad.append(f"misaligned buffer: status {e.status}")
        if not torch.equal(part, base):
            bad.append("refused call wrote")
        return desc, bad
    dp.dp_add_noise_slice(part, first, sigma, C_, scale, seed, tid, step)
    torch.cuda.synchronize()
    z = NO.standard_normals(n, seed, tid, step, start=first)
    want = scale * (base.cpu().numpy().astype(np.float64) + sigma * C_ * z)
    e = np.abs(part.cpu().numpy() - want).max()
    if not e < 1e-6 * max(1.0, sigma * C_ * scale) + 2e-7 * np.abs(want).max():
        bad.append(f"noise err {e:.3e}")
    rest = torch.cat([buf[:off], buf[off + n:]])
    if not torch.isfinite(rest).all():
        bad.append("neighbours damaged")
    return desc, bad


def fused_noise_case(rng, k):
    """grouped clipped sums with the noise drawn in the same call == plain sums + dp_add_noise"""
    B = int(rng.integers(1, 5))
    T = pick(rng, [16, 64, 100, 128, 200, 256])
    n = int(rng.integers(1, 4))
    lays, shapes = [], []
    for _ in range(n):
        d, p = rand_dim(rng), rand_dim(rng)
        if int(rng.integers(4)) == 0:
            p = pick(rng, [128 * 40, 128 * 100])             # enough tiles for the epilogue path
        lda = W.round_up(d, 8) if d % 8 else None
        ldg = W.round_up(p, 8) if p % 8 else None
        A = W._normal((B, T, d), 1.0, "bf16", int(rng.integers(1 << 60)), ld=lda)
        G = W._normal((B, T, p), 1e-2, "bf16", int(rng.integers(1 << 60)), ld=ldg)
        lays.append(dp.Linear(P.to_device(A), P.to_device(G), d=d, p=p))
        shapes.append((d, p))
    desc = f"#{k} fused noise B{B} T{T} " + " ".join(f"{d}x{p}" for d, p in shapes)
    bad = []
    sq = torch.full((B,), float(rng.uniform(0.5, 8.0)), device=_dev())
    tids = [int(rng.integers(0, 1000)) for _ in shapes]
    seed, step = int(rng.integers(1 << 62)), int(rng.integers(1 << 20))
    sigma, C_, scale = 0.8, float(rng.uniform(0.5, 2.0)), pick(rng, [1.0, 0.25])
    fused = [torch.empty(p, d, device=_dev()) for d, p in shapes]
    dp.dp_clip_accumulate_noise_grouped(lays, B, T, sq, C_, fused, sigma, scale, seed, tids, step)
    plain = [torch.empty(p, d, device=_dev()) for d, p in shapes]
    dp.dp_clip_accumulate_grouped(lays, B, T, sq, C_, plain)
    sums = [t.clone() for t in plain]
    torch.cuda.synchronize()
    for f, s0, tid, (d, p) in zip(fused, sums, tids, shapes):
        want = NO.add_noise(s0.cpu().numpy().astype(np.float64), sigma, C_, scale, seed, tid, step)
        e = np.abs(f.cpu().numpy() - want).max()
        if not e < 1e-6 * max(1.0, C_) + 1e-6 * np.abs(want).max():
            bad.append(f"{d}x{p} err {e:.3e}")
    return desc, bad


def vector_case(rng, k):
    dtype = pick(rng, ["bf16", "f32"])
    B = int(rng.integers(1, 6))
    T = pick(rng, [1, 16, 37, 100, 128, 300, 512])
    n = int(rng.integers(1, 4))
    prm, hosts = [], []
    g_std = 1.0 if dtype == "f32" else 1e-2
    for _ in range(n):
        p = rand_dim(rng)
        with_x = bool(rng.integers(2))
        G = W._normal((B, T, p), g_std, dtype, int(rng.integers(1 << 60)))
        X = W._normal((B, T, p), 1.0, dtype, int(rng.integers(1 << 60))) if with_x else None
        prm.append(dp.Vector(P.to_device(G), P.to_device(X) if with_x else None, p=p))
        hosts.append((G.widened(), X.widened() if with_x else None, p))
    desc = f"#{k} vectors {dtype} B{B} T{T} " + " ".join(str(p) + ("x" if x is not None else "") for _, x, p in hosts)
    bad = []
    sq = torch.zeros(B, device=_dev())
    dp.dp_vector_norms(prm, B, T, sq)
    torch.cuda.synchronize()
    want = sum(O.vector_sq_norms(g, x) for g, x, _ in hosts)
    e = rel(sq.cpu().numpy(), want).max()
    if not e < (1e-4 if dtype == "f32" else 2e-3):
        bad.append(f"norm err {e:.3e}")
    Cc = float(np.median(np.sqrt(want)))
    sq_in = torch.from_numpy(want.astype(np.float32)).to(_dev())
    _, R = O.clip_factors(sq_in.cpu().numpy().astype(np.float64), Cc)
    beta = pick(rng, [0.0, 1.0])
    outs0 = [torch.randn(p, device=_dev()) for _, _, p in hosts]
    outs = [o.clone() for o in outs0]
    dp.dp_clip_accumulate_vectors(prm, B, T, sq_in, Cc, outs, beta=beta)
    torch.cuda.synchronize()
    for (g, x, p), o, o0 in zip(hosts, outs, outs0):
        w = O.clipped_sum_vector(g, x, R) + beta * o0.cpu().numpy().astype(np.float64)
        fe = frob_rel(o.cpu().numpy(), w)
        if not fe < 1e-5:
            bad.append(f"sum err p{p} {fe:.3e}")
    return desc, bad


@pytest.mark.parametrize("case,n,seed", [(linear_case, 200, 101), (grouped_case, 80, 102),
                                          (embed_case, 80, 103), (cross_case, 60, 104),
                                          (noise_case, 150, 105), (fused_noise_case, 40, 106),
                                          (vector_case, 80, 107)])
def test_random_shapes_against_the_oracle(case, n, seed):
    rng = np.random.default_rng(seed)
    failures = []
    for k in range(n):
        desc, bad = case(rng, k)
        if bad:
            failures.append((desc, bad))
    assert not failures, failures
