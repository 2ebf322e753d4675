"""GPU parity: every C-ABI entry point against the float64 CPU oracle on the same seeded inputs.

Tolerances (from the benchmark spec): per-example norms and clip factors 1e-4 relative for fp32
inputs, 1e-2 relative for bf16 inputs with fp32 accumulation; clipped sums 1e-2 relative
Frobenius error; integer outputs bit-exact; noise 1e-6 absolute per element.  Because both sides
start from the same bf16 values, the kernels land far inside the bf16 bound; the tests assert a
tighter 2e-3 there so that a wrong tile or a dropped K step cannot hide under the tolerance.
"""
import numpy as np
import pytest
import torch

from oracle import dp_oracle as O
from oracle import noise_oracle as NO
from paper_2609_40335_b200 import binding as dp
from paper_2609_40335_b200 import pipeline as P
from paper_2609_40335_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 1e-2
TIGHT_BF16 = 2e-3
TOL_SUM = 1e-2


def dev():
    return torch.device("cuda:0")


def rel(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return np.abs(a - b) / np.maximum(np.abs(b), 1e-300)


def frob_rel(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def host_linear(B, T, d, p, dtype, seed, a_std=1.0, g_std=1e-2, ldg=None):
    rng = np.random.default_rng(seed)
    A = W._normal((B, T, d), a_std, dtype, int(rng.integers(1 << 60)))
    G = W._normal((B, T, p), g_std, dtype, int(rng.integers(1 << 60)), ld=ldg)
    return A, G


def dev_linear(A, G, mode=dp.DP_NORM_AUTO):
    return dp.Linear(P.to_device(A), P.to_device(G), d=A.cols, p=G.cols, mode=mode)


def check_status(ds_status):
    assert int(ds_status.item()) == 0


# ------------------------------------------------------------------ config 1, end to end
def test_cfg1_end_to_end_fp32():
    w = W.named_workload("cfg1")
    ds = P.upload(w)
    P.dp_step(ds, seed=0, step=0, noise=False)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    lin = [(l.A.widened(), l.G.widened()) for l in w.linears]
    ref = O.dp_step(lin, w.ids, w.G_emb.widened(), w.V, w.C)
    assert rel(ds.sq.cpu().numpy(), ref["sq"]).max() < TOL_F32
    assert rel(ds.norms.cpu().numpy(), ref["norms"]).max() < TOL_F32
    assert rel(ds.clip.cpu().numpy(), ref["clip"]).max() < TOL_F32
    assert frob_rel(ds.outs["linear0"].cpu().numpy(), ref["sums"]["linear0"]) < 1e-5
    assert frob_rel(ds.outs["wte"].cpu().numpy(), ref["sums"]["wte"]) < 1e-5
    # noised clipped sum: same stream convention as the oracle
    before = {k: v.clone() for k, v in ds.outs.items()}
    P.noise_phase(ds, seed=0, step=0)
    torch.cuda.synchronize()
    for tid, name in enumerate(sorted(ds.outs)):
        want = NO.add_noise(before[name].cpu().numpy().astype(np.float64), w.sigma, w.C, 1.0, 0, tid, 0)
        got = ds.outs[name].cpu().numpy()
        assert np.abs(got - want).max() < 2e-6 + 1e-6 * np.abs(want).max()


# ------------------------------------------------------------------ linear-layer norms
GHOST_CASES = [
    # B, T, d, p, ld padding of G
    (3, 128, 768, 256, None),       # one tile, the HBM-bound regime
    (2, 100, 72, 136, None),        # ragged T, K tails not multiples of 64
    (2, 200, 192, 320, None),       # two row tiles with a ragged second one (3 tile pairs)
    (1, 384, 128, 64, None),        # three row tiles (6 tile pairs)
    (2, 128, 256, 5003, 5008),      # wide operand split across CTAs, odd width, NaN padding
    (5, 16, 64, 64, None),          # tiny T
    (1, 1, 64, 128, None),          # single token: Eq. 5
]


@pytest.mark.parametrize("B,T,d,p,ldg", GHOST_CASES)
@pytest.mark.parametrize("mode", [dp.DP_NORM_GHOST, dp.DP_NORM_DIRECT])
def test_linear_norms_bf16_tensor_core(B, T, d, p, ldg, mode):
    A, G = host_linear(B, T, d, p, "bf16", seed=B * 1000 + T + d + p, ldg=ldg)
    lin = dev_linear(A, G, mode)
    sq = torch.zeros(B, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    used = dp.dp_ghost_norms([lin], B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    assert used == [mode]
    want = O.linear_sq_norms(A.widened(), G.widened())
    got = sq.cpu().numpy()
    assert np.isfinite(got).all()
    assert rel(got, want).max() < TIGHT_BF16, (got, want)
    # accumulation semantics: a second call adds the same amount
    dp.dp_ghost_norms([lin], B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    assert rel(sq.cpu().numpy(), 2 * want).max() < TIGHT_BF16


def test_linear_norms_grouped_layers_and_auto_rule():
    B, T = 4, 128
    shapes = [(768, 2304), (768, 768), (768, 3072), (3072, 768), (64, 64)]
    host = [host_linear(B, T, d, p, "bf16", seed=77 + k) for k, (d, p) in enumerate(shapes)]
    layers = [dev_linear(A, G) for A, G in host]
    sq = torch.zeros(B, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    used = dp.dp_ghost_norms(layers, B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    # AUTO: direct iff T*T > d*p (only the 64x64 layer: 16384 > 4096)
    assert used == [dp.DP_NORM_GHOST] * 4 + [dp.DP_NORM_DIRECT]
    want = sum(O.linear_sq_norms(A.widened(), G.widened()) for A, G in host)
    assert rel(sq.cpu().numpy(), want).max() < TIGHT_BF16
    # deterministic: same inputs, bitwise-equal result
    sq2 = torch.zeros(B, device=dev())
    dp.dp_ghost_norms(layers, B, T, sq2, dev_status=st)
    torch.cuda.synchronize()
    assert torch.equal(sq, sq2)


def test_tensor_core_and_fma_paths_agree_on_device():
    B, T, d, p = 8, 256, 768, 768
    A, G = host_linear(B, T, d, p, "bf16", seed=5)
    lin = dev_linear(A, G, dp.DP_NORM_GHOST)
    sq_tc = torch.zeros(B, device=dev())
    dp.dp_ghost_norms([lin], B, T, sq_tc)
    prev = dp.dp_debug_force_fma(True)
    try:
        sq_fma = torch.zeros(B, device=dev())
        dp.dp_ghost_norms([lin], B, T, sq_fma)
    finally:
        dp.dp_debug_force_fma(prev)
    torch.cuda.synchronize()
    assert rel(sq_tc.cpu().numpy(), sq_fma.cpu().numpy()).max() < 1e-4


@pytest.mark.parametrize("mode", [dp.DP_NORM_GHOST, dp.DP_NORM_DIRECT])
def test_linear_norms_fp32(mode):
    B, T, d, p = 3, 21, 40, 33
    A, G = host_linear(B, T, d, p, "f32", seed=9, g_std=1.0)
    lin = dev_linear(A, G, mode)
    sq = torch.zeros(B, device=dev())
    dp.dp_ghost_norms([lin], B, T, sq)
    torch.cuda.synchronize()
    assert rel(sq.cpu().numpy(), O.linear_sq_norms(A.widened(), G.widened())).max() < TOL_F32


# ------------------------------------------------------------------------ clipped sums
ACC_CASES = [
    # B, T, d, p
    (4, 128, 768, 768),      # few tiles: K split across CTAs
    (3, 100, 200, 300),      # ragged T, M and N tails inside a tile
    (2, 64, 1024, 128),      # several N tiles
    (6, 16, 64, 64),         # tiny T (a K step is mostly zero fill)
    (2, 128, 256, 1003),     # odd M (LM-head like), padded ld
]


@pytest.mark.parametrize("B,T,d,p", ACC_CASES)
@pytest.mark.parametrize("beta", [0.0, 1.0])
def test_clip_accumulate_bf16_tensor_core(B, T, d, p, beta):
    ldg = W.round_up(p, 8)
    A, G = host_linear(B, T, d, p, "bf16", seed=B + T + d + p, ldg=ldg if ldg != p else None)
    sq_true = O.linear_sq_norms(A.widened(), G.widened())
    Cc = float(np.median(np.sqrt(sq_true)))              # some examples clipped, some not
    sq = torch.from_numpy(sq_true.astype(np.float32)).to(dev())
    out0 = torch.randn(p, d, device=dev())
    out = out0.clone()
    clip = torch.zeros(B, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_clip_accumulate(P.to_device(A), P.to_device(G), sq, Cc, out, beta=beta, d=d, p=p, clip=clip,
                          dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    _, R = O.clip_factors(sq.cpu().numpy().astype(np.float64), Cc)
    assert (R < 1).any() and (R == 1).any()
    assert rel(clip.cpu().numpy(), R).max() < 1e-6
    want = O.clipped_sum_linear(A.widened(), G.widened(), R) + beta * out0.cpu().numpy().astype(np.float64)
    assert frob_rel(out.cpu().numpy(), want) < TOL_SUM
    assert frob_rel(out.cpu().numpy(), want) < 5e-3      # bf16 rounding of R*g only


def test_clip_accumulate_grouped_matches_per_layer_calls_and_oracle():
    B, T = 4, 128
    shapes = [(768, 2304), (768, 768), (200, 136), (3072, 768)]
    host = [host_linear(B, T, d, p, "bf16", seed=300 + k) for k, (d, p) in enumerate(shapes)]
    layers = [dev_linear(A, G) for A, G in host]
    sq_true = sum(O.linear_sq_norms(A.widened(), G.widened()) for A, G in host)
    Cc = float(np.median(np.sqrt(sq_true)))
    sq = torch.from_numpy(sq_true.astype(np.float32)).to(dev())
    outs = [torch.empty(p, d, device=dev()) for d, p in shapes]
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_clip_accumulate_grouped(layers, B, T, sq, Cc, outs, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    _, R = O.clip_factors(sq.cpu().numpy().astype(np.float64), Cc)
    for (A, G), l, o in zip(host, layers, outs):
        want = O.clipped_sum_linear(A.widened(), G.widened(), R)
        assert frob_rel(o.cpu().numpy(), want) < 5e-3
        single = torch.empty_like(o)
        dp.dp_clip_accumulate(l.A, l.G, sq, Cc, single, d=l.d, p=l.p)
        torch.cuda.synchronize()
        assert frob_rel(single.cpu().numpy(), want) < 5e-3


def test_clip_accumulate_unclipped_is_plain_gemm_and_deterministic():
    B, T, d, p = 4, 128, 256, 384
    A, G = host_linear(B, T, d, p, "bf16", seed=3)
    sq = torch.full((B,), 1e-12, device=dev())            # norms far below C: every R_i = 1
    out = torch.empty(p, d, device=dev())
    dp.dp_clip_accumulate(P.to_device(A), P.to_device(G), sq, 1.0, out)
    out2 = torch.empty(p, d, device=dev())
    dp.dp_clip_accumulate(P.to_device(A), P.to_device(G), sq, 1.0, out2)
    torch.cuda.synchronize()
    want = G.widened().reshape(B * T, p).T @ A.widened().reshape(B * T, d)
    assert frob_rel(out.cpu().numpy(), want) < 1e-5       # no rescaling: fp32 accumulation only
    assert torch.equal(out, out2)


def test_clip_accumulate_fp32():
    B, T, d, p = 3, 10, 70, 50
    A, G = host_linear(B, T, d, p, "f32", seed=4, g_std=1.0)
    sq_true = O.linear_sq_norms(A.widened(), G.widened())
    Cc = float(np.median(np.sqrt(sq_true)))
    sq = torch.from_numpy(sq_true.astype(np.float32)).to(dev())
    out = torch.empty(p, d, device=dev())
    dp.dp_clip_accumulate(P.to_device(A), P.to_device(G), sq, Cc, out)
    torch.cuda.synchronize()
    _, R = O.clip_factors(sq.cpu().numpy().astype(np.float64), Cc)
    assert frob_rel(out.cpu().numpy(), O.clipped_sum_linear(A.widened(), G.widened(), R)) < 1e-5


# --------------------------------------------------------------------------- embeddings
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,d,V,dist", [(4, 16, 64, 1000, "uniform"), (3, 128, 768, 50257, "zipf"),
                                          (2, 300, 200, 50257, "zipf"), (2, 40, 768, 7, "uniform"),
                                          (2, 33, 10, 5, "uniform")])
def test_embed_norms_and_first_occurrence(dtype, B, T, d, V, dist):
    ids = W.zipf_ids(B, T, V, 1.1, 11) if dist == "zipf" else W.uniform_ids(B, T, V, 11)
    ids[0, :] = ids[0, 0]                                  # one example: a single repeated token
    G = W._normal((B, T, d), 1.0 if dtype == "f32" else 1e-2, dtype, 12)
    sq = torch.zeros(B, device=dev())
    fo = torch.full((B, T), -1, dtype=torch.int32, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_embed_norms(torch.from_numpy(ids).to(dev()), P.to_device(G), V, sq, first_occ=fo, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    np.testing.assert_array_equal(fo.cpu().numpy(), O.first_occurrence(ids))
    tol = TOL_F32 if dtype == "f32" else TIGHT_BF16
    assert rel(sq.cpu().numpy(), O.embed_sq_norms(ids, G.widened(), V)).max() < tol


def test_embed_norms_position_table_and_bad_ids():
    B, T, d = 2, 50, 96
    G = W._normal((B, T, d), 1e-2, "bf16", 13)
    pos = np.broadcast_to(np.arange(T, dtype=np.int32), (B, T)).copy()
    sq = torch.zeros(B, device=dev())
    dp.dp_embed_norms(torch.from_numpy(pos).to(dev()), P.to_device(G), T, sq)
    torch.cuda.synchronize()
    assert rel(sq.cpu().numpy(), (G.widened() ** 2).sum(axis=(1, 2))).max() < TIGHT_BF16
    # out-of-range ids are flagged and skipped
    bad = pos.copy()
    bad[1, 7] = T + 3
    bad[1, 9] = -1
    sq.zero_()
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_embed_norms(torch.from_numpy(bad).to(dev()), P.to_device(G), T, sq, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) & dp.DP_DEV_BAD_ID
    g = G.widened()
    want1 = (g[1] ** 2).sum() - (g[1, 7] ** 2).sum() - (g[1, 9] ** 2).sum()
    assert rel(sq.cpu().numpy()[1], want1) < TIGHT_BF16


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,d,V,beta", [(4, 16, 64, 1000, 0.0), (3, 128, 768, 50257, 0.0),
                                          (5, 700, 100, 300, 1.0), (2, 40, 132, 7, 1.0)])
def test_clip_accumulate_embed(dtype, B, T, d, V, beta):
    ids = W.zipf_ids(B, T, V, 1.1, 21)
    G = W._normal((B, T, d), 1.0 if dtype == "f32" else 1e-2, dtype, 22)
    sq_true = O.embed_sq_norms(ids, G.widened(), V)
    Cc = float(np.median(np.sqrt(sq_true)))
    sq = torch.from_numpy(sq_true.astype(np.float32)).to(dev())
    out0 = torch.randn(V, d, device=dev())
    out = out0.clone()
    perm = torch.full((B * T,), -1, dtype=torch.int32, device=dev())
    seg = torch.full((V + 1,), -1, dtype=torch.int32, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_clip_accumulate_embed(torch.from_numpy(ids).to(dev()), P.to_device(G), V, sq, Cc, out, beta=beta,
                                perm=perm, seg=seg, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    want_perm, want_seg = O.stable_token_sort(ids, V)
    np.testing.assert_array_equal(perm.cpu().numpy(), want_perm)
    np.testing.assert_array_equal(seg.cpu().numpy(), want_seg)
    _, R = O.clip_factors(sq.cpu().numpy().astype(np.float64), Cc)
    want = O.clipped_sum_embed(ids, G.widened(), R, V) + beta * out0.cpu().numpy().astype(np.float64)
    assert frob_rel(out.cpu().numpy(), want) < 1e-5
    if beta == 0.0:
        untouched = np.setdiff1d(np.arange(V), ids.reshape(-1))
        assert (out.cpu().numpy()[untouched] == 0).all()


# --------------------------------------------------------------------------- tied cross term
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,d,V", [(3, 16, 64, 1000), (2, 128, 768, 50257), (2, 70, 100, 33),
                                     (2, 300, 136, 4099)])
def test_tied_cross_term(dtype, B, T, d, V):
    g_std = 1.0 if dtype == "f32" else 1e-2
    ids = W.zipf_ids(B, T, V, 1.1, 31)
    ldd = W.round_up(d, 8) if (dtype == "bf16" and d % 8) else None     # TMA pitch, NaN padding
    G_emb = W._normal((B, T, d), g_std, dtype, 32, ld=ldd)
    A_lm = W._normal((B, T, d), 1.0, dtype, 33, ld=ldd)
    ld = W.round_up(V, 8) if dtype == "bf16" else V
    G_lm = W._normal((B, T, V), g_std, dtype, 34, ld=ld if ld != V else None)
    ref = O.tied_sq_norms(ids, G_emb.widened(), A_lm.widened(), G_lm.widened(), V)
    sq = torch.zeros(B, device=dev())
    cross = torch.zeros(B, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_tied_cross_term(torch.from_numpy(ids).to(dev()), P.to_device(G_emb), P.to_device(A_lm),
                          P.to_device(G_lm), V, sq=sq, cross=cross, d=d, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    scale = np.sqrt(ref["in"] * ref["out"])               # the term's natural scale (Cauchy-Schwarz)
    tol = TOL_F32 if dtype == "f32" else TIGHT_BF16
    assert (np.abs(cross.cpu().numpy() - ref["cross"]) / scale).max() < tol
    assert (np.abs(sq.cpu().numpy() - 2 * ref["cross"]) / scale).max() < tol


# ---------------------------------------------------------------------------------- noise
@pytest.mark.parametrize("n", [1, 3, 4, 1023, 1 << 20])
def test_noise_matches_oracle_stream(n):
    seed, tid, step = (0xABCDEF12 << 32) | 0x3456789A, 5, 17
    x = torch.zeros(n, device=dev())
    dp.dp_add_noise(x, 1.0, 1.0, 1.0, seed, tid, step)
    torch.cuda.synchronize()
    want = NO.standard_normals(n, seed, tid, step)
    assert np.abs(x.cpu().numpy() - want).max() < 1e-6


def test_noise_tail_region_and_scaling():
    n = 1 << 24                                            # ~60 thousand values beyond |z| = 3.3 pass through
    x = torch.zeros(n, device=dev())
    dp.dp_add_noise(x, 1.0, 1.0, 1.0, 7, 0, 0)
    z = NO.standard_normals(n, 7, 0, 0)
    got = x.cpu().numpy()
    assert np.abs(got - z).max() < 1e-6
    assert np.abs(z).max() > 4.5
    base = torch.randn(4096, device=dev())
    y = base.clone()
    dp.dp_add_noise(y, 0.8, 0.5, 0.25, 7, 1, 2)
    want = NO.add_noise(base.cpu().numpy(), 0.8, 0.5, 0.25, 7, 1, 2)
    assert np.abs(y.cpu().numpy() - want).max() < 1e-6
    y2 = base.clone()
    dp.dp_add_noise(y2, 0.8, 0.5, 0.25, 7, 1, 2)
    assert torch.equal(y, y2)
    y3 = base.clone()
    dp.dp_add_noise(y3, 0.0, 1.0, 1.0, 7, 1, 2)
    assert torch.equal(y3, base)


# ------------------------------------------------------------------ fused noise
@pytest.mark.parametrize("shapes", [
    [(768, 128 * 100), (768, 768)],      # enough tiles: noise drawn in the GEMM epilogue
    [(256, 384)],                        # few tiles: K split, noise after the reduce
    [(50, 128 * 80), (104, 200)],        # widths not a multiple of 4: quads straddle rows
])
def test_fused_noise_in_gemm_equals_unfused_calls(shapes):
    B, T = 4, 128
    host = [host_linear(B, T, d, p, "bf16", seed=500 + k, ldg=W.round_up(p, 8) if p % 8 else None)
            for k, (d, p) in enumerate(shapes)]
    layers = []
    for (A, G), (d, p) in zip(host, shapes):
        if d % 8:                                           # pad the activation pitch for TMA
            a = torch.zeros(B, T, W.round_up(d, 8), dtype=torch.bfloat16, device=dev())
            a[:, :, :d] = P.to_device(A)
            layers.append(dp.Linear(a, P.to_device(G), d=d, p=p))
        else:
            layers.append(dev_linear(A, G))
    sq = torch.full((B,), 4.0, device=dev())
    tids = [7 + k for k in range(len(shapes))]
    seed, step, sigma, C_, scale = 99, 3, 0.8, 1.0, 0.25
    fused = [torch.empty(p, d, device=dev()) for d, p in shapes]
    dp.dp_clip_accumulate_noise_grouped(layers, B, T, sq, C_, fused, sigma, scale, seed, tids, step)
    plain = [torch.empty(p, d, device=dev()) for d, p in shapes]
    dp.dp_clip_accumulate_grouped(layers, B, T, sq, C_, plain)
    sums = [t.clone() for t in plain]
    for t, tid in zip(plain, tids):
        dp.dp_add_noise(t, sigma, C_, scale, seed, tid, step)
    torch.cuda.synchronize()
    for f, u, s0, tid in zip(fused, plain, sums, tids):
        assert torch.equal(f, u)                            # same stream, same arithmetic
        want = NO.add_noise(s0.cpu().numpy().astype(np.float64), sigma, C_, scale, seed, tid, step)
        assert np.abs(f.cpu().numpy() - want).max() < 1e-6


@pytest.mark.parametrize("beta", [0.0, 1.0])
def test_fused_noise_in_embedding_matches_unfused_calls(beta):
    B, T, d, V = 3, 128, 768, 5003
    ids = W.zipf_ids(B, T, V, 1.1, 41)
    G = W._normal((B, T, d), 1e-2, "bf16", 42)
    sq = torch.full((B,), 9.0, device=dev())
    base = torch.randn(V, d, device=dev())
    seed, tid, step, sigma, C_, scale = 5, 2, 1, 0.8, 1.0, 0.5
    dids, dG = torch.from_numpy(ids).to(dev()), P.to_device(G)
    fused = base.clone()
    dp.dp_clip_accumulate_embed_noise(dids, dG, V, sq, C_, fused, sigma, scale, seed, tid, step, beta=beta)
    plain = base.clone()
    dp.dp_clip_accumulate_embed(dids, dG, V, sq, C_, plain, beta=beta)
    if beta == 0.0:
        dp.dp_add_noise(plain, sigma, C_, scale, seed, tid, step)
    else:
        # tied case: the table already holds noise + head; the call adds scale * row sums
        plain = base + scale * (plain - base)
    torch.cuda.synchronize()
    assert torch.allclose(fused, plain, rtol=1e-5, atol=2e-6)


def test_fused_and_unfused_steps_agree():
    w = W.named_workload("cfg4", B=3, n_blocks=1, V=4099)
    a, b = P.upload(w), P.upload(w)
    c = P.upload(w)
    P.dp_step(a, seed=11, step=2, fused=True)                      # noise prefill on a side stream
    P.dp_step(b, seed=11, step=2, fused=False)
    P.dp_step(c, seed=11, step=2, fused=True, overlap=False)
    torch.cuda.synchronize()
    check_status(a.dev_status)
    for k in a.outs:
        assert torch.allclose(a.outs[k], b.outs[k], rtol=1e-5, atol=2e-6), k
        assert torch.allclose(c.outs[k], b.outs[k], rtol=1e-5, atol=2e-6), k


def test_overlapped_step_untied_with_positions_matches_unfused():
    w = W.named_workload("cfg3", B=2, T=256, n_blocks=1, V=3001)
    a, b = P.upload(w), P.upload(w)
    for step in range(2):                                          # twice: side-stream reuse
        P.dp_step(a, seed=5, step=step, fused=True)
        P.dp_step(b, seed=5, step=step, fused=False)
    torch.cuda.synchronize()
    for k in a.outs:
        assert torch.allclose(a.outs[k], b.outs[k], rtol=1e-5, atol=2e-6), k


def test_noise_fp32_path_error_bound_exhaustive():
    """The fp32 Box-Muller path is used up to r^2 = threshold; beyond it float64 takes over.  An
    exhaustive device scan of both fp32 factors against float64 (all 2^24 inputs each) must keep
    the worst-case error of z = r * cos/sin below the 1e-6 tolerance at that threshold."""
    L = dp.load()
    out = torch.zeros(4, dtype=torch.float64, device=dev())
    assert L.dp_debug_noise_error_scan(0.0, out.data_ptr(), None) == 0
    torch.cuda.synchronize()
    err_r, err_dir, r_max, thr = out.tolist()
    assert 3.3 ** 2 <= thr <= 34.0 and r_max <= thr ** 0.5 + 1e-6
    bound = (err_r + err_dir + 2.0 ** -24) * r_max          # relative r, absolute direction, product rounding
    assert bound < 1e-6, (err_r, err_dir, r_max, bound)


# ---------------------------------------------------------------------------- error paths
def test_argument_errors_are_reported_before_any_launch():
    B, T, d, p = 2, 16, 64, 64
    A, G = host_linear(B, T, d, p, "bf16", seed=1)
    a, g = P.to_device(A), P.to_device(G)
    sq = torch.zeros(B, device=dev())
    with pytest.raises(dp.DpGhostError) as e:
        dp.dp_ghost_norms([dp.Linear(a[:, :, 1:], g, d=d - 1)], B, T, sq)    # misaligned base
    assert e.value.status == 3
    with pytest.raises(dp.DpGhostError) as e:
        dp.dp_ghost_norms([dp.Linear(a, g, mode=7)], B, T, sq)
    assert e.value.status == 1
    with pytest.raises(dp.DpGhostError) as e:
        dp.dp_ghost_norms([dp.Linear(a, g)], B, T, sq, ws=torch.empty(4, dtype=torch.uint8, device=dev()))
    assert e.value.status == 4
    out = torch.empty(p, d, device=dev())
    with pytest.raises(dp.DpGhostError) as e:
        dp.dp_clip_accumulate(a, g, sq, 1.0, out, beta=0.5)
    assert e.value.status == 1
    with pytest.raises(dp.DpGhostError) as e:
        dp.dp_clip_accumulate(a, g, sq, -1.0, out)
    assert e.value.status == 1
    with pytest.raises(dp.DpGhostError) as e:
        dp.dp_add_noise(out.view(-1)[1:], 1.0, 1.0, 1.0, 0, 0, 0)          # not 16-byte aligned
    assert e.value.status == 3
    with pytest.raises(dp.DpGhostError):
        dp.dp_add_noise(torch.zeros(4), 1.0, 1.0, 1.0, 0, 0, 0)            # host tensor: no CPU path
    torch.cuda.synchronize()
    assert float(sq.abs().sum()) == 0.0


# ------------------------------------------------------------- reduced model-shaped steps
@pytest.mark.parametrize("name,over", [
    ("cfg2", dict(B=4, n_blocks=1, V=5003)),
    ("cfg3", dict(B=2, T=256, n_blocks=1, V=3001)),
    ("cfg4", dict(B=3, n_blocks=1, V=4099)),
])
def test_reduced_model_step_matches_oracle(name, over):
    w = W.named_workload(name, **over)
    ds = P.upload(w)
    P.dp_step(ds, noise=False)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    lin = [(l.A.widened(), l.G.widened()) for l in w.linears]
    ref = O.dp_step(lin, w.ids, w.G_emb.widened(), w.V, w.C, lm=(w.lm.A.widened(), w.lm.G.widened()),
                    tied=w.tied, positions=w.positions)
    assert rel(ds.sq.cpu().numpy(), ref["sq"]).max() < TIGHT_BF16
    assert rel(ds.clip.cpu().numpy(), ref["clip"]).max() < TIGHT_BF16
    if w.tied:
        scale = np.sqrt(ref["sq_in"] * ref["sq_out"])
        assert (np.abs(ds.cross.cpu().numpy() - ref["cross"]) / scale).max() < TIGHT_BF16
    for k, want in ref["sums"].items():
        got = ds.outs[k].cpu().numpy()
        if k == "wpe":
            assert (got[w.T:] == 0).all()
            got = got[: w.T]
        assert frob_rel(got, want) < TOL_SUM, k


# ------------------------------------------------------ full-size cfg2, sampled outputs
def test_cfg2_full_size_sampled_against_oracle():
    """The bench configuration itself (DistilGPT2 shape, B=32, T=128, 24 linears + LM head with
    V=50257, one grouped launch per phase).  The oracle is too slow for all of it, so it checks
    (a) the per-example norms of three sampled examples over every layer, and (b) the clipped
    sums of sampled layers and sampled LM-head rows, with per-example squared norms drawn by
    the test (they are an input of the clipped-sum calls)."""
    w = W.named_workload("cfg2")
    ds = P.upload(w)
    P.norms_phase(ds)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    sq_gpu = ds.sq.cpu().numpy()
    for i in (0, 13, 31):
        sl = slice(i, i + 1)
        lin = [(l.A.widened_rows(sl), l.G.widened_rows(sl)) for l in w.linears]
        ref = O.dp_step(lin, w.ids[sl], w.G_emb.widened_rows(sl), w.V, w.C,
                        lm=(w.lm.A.widened_rows(sl), w.lm.G.widened_rows(sl)), want_sums=False)
        assert abs(sq_gpu[i] - ref["sq"][0]) / ref["sq"][0] < TIGHT_BF16, i
    # clipped sums with test-chosen norms: half of the examples clipped
    rng = np.random.default_rng(123)
    sq_in = (rng.uniform(0.25, 4.0, w.B) ** 2).astype(np.float32)
    ds.sq.copy_(torch.from_numpy(sq_in))
    P.clip_phase(ds)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    _, R = O.clip_factors(sq_in.astype(np.float64), w.C)
    assert (R < 1).any() and (R == 1).any()
    for k in (0, 1, 10, 23):                                  # one of each layer shape
        l = w.linears[k]
        want = O.clipped_sum_linear(l.A.widened(), l.G.widened(), R)
        assert frob_rel(ds.outs[f"linear{k}"].cpu().numpy(), want) < 5e-3, k
    rows = np.array([0, 1, 127, 128, 255, 256, 25000, 50175, 50176, 50255, 50256])
    Gs = W.bf16_bits_to_f32(w.lm.G.data[:, :, rows]).astype(np.float64)
    want = O.clipped_sum_linear(w.lm.A.widened(), Gs, R)
    got = ds.outs["lm_head"].cpu().numpy()[rows]
    assert frob_rel(got, want) < 5e-3
    want_e = O.clipped_sum_embed(w.ids, w.G_emb.widened(), R, w.V)
    assert frob_rel(ds.outs["wte"].cpu().numpy(), want_e) < 1e-5


# ------------------------------------------------------ bias / LayerNorm parameters
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,p,with_x", [(3, 128, 768, True), (2, 100, 300, False), (4, 37, 2304, True),
                                          (2, 16, 10, True), (5, 300, 1000, False)])
def test_vector_parameter_norms_and_clipped_sums(dtype, B, T, p, with_x):
    g_std = 1.0 if dtype == "f32" else 1e-2
    G = W._normal((B, T, p), g_std, dtype, 61)
    X = W._normal((B, T, p), 1.0, dtype, 62) if with_x else None
    Gw, Xw = G.widened(), (X.widened() if with_x else None)
    prm = [dp.Vector(P.to_device(G), P.to_device(X) if with_x else None, p=p)]
    sq = torch.zeros(B, device=dev())
    dp.dp_vector_norms(prm, B, T, sq)
    torch.cuda.synchronize()
    sq_true = O.vector_sq_norms(Gw, Xw)
    tol = TOL_F32 if dtype == "f32" else TIGHT_BF16
    assert rel(sq.cpu().numpy(), sq_true).max() < tol
    Cc = float(np.median(np.sqrt(sq_true)))
    sq_in = torch.from_numpy(sq_true.astype(np.float32)).to(dev())
    _, R = O.clip_factors(sq_in.cpu().numpy().astype(np.float64), Cc)
    base = torch.randn(p, device=dev())
    for beta in (0.0, 1.0):
        out = base.clone()
        dp.dp_clip_accumulate_vectors(prm, B, T, sq_in, Cc, [out], beta=beta)
        torch.cuda.synchronize()
        want = O.clipped_sum_vector(Gw, Xw, R) + beta * base.cpu().numpy().astype(np.float64)
        assert frob_rel(out.cpu().numpy(), want) < 1e-5
    # fused Gaussian mechanism == clipped sum followed by dp_add_noise, same stream
    fused, plain = torch.empty(p, device=dev()), torch.empty(p, device=dev())
    dp.dp_clip_accumulate_vectors(prm, B, T, sq_in, Cc, [fused], noise=(0.8, 0.5, 77, [9], 4))
    dp.dp_clip_accumulate_vectors(prm, B, T, sq_in, Cc, [plain])
    if p % 4 == 0:
        dp.dp_add_noise(plain, 0.8, Cc, 0.5, 77, 9, 4)
        torch.cuda.synchronize()
        assert torch.equal(fused, plain)
    want = NO.add_noise(O.clipped_sum_vector(Gw, Xw, R), 0.8, Cc, 0.5, 77, 9, 4)
    torch.cuda.synchronize()
    assert np.abs(fused.cpu().numpy() - want).max() < 1e-6 + 1e-5 * np.abs(want).max()


def test_full_model_step_with_biases_and_layernorm_matches_oracle():
    w = W.named_workload("cfg3", B=2, T=128, n_blocks=2, V=3001, full_model=True)
    assert len(w.vectors) == 2 * (4 + 4) + 2
    ds = P.upload(w)
    P.dp_step(ds, noise=False)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    lin = [(l.A.widened(), l.G.widened()) for l in w.linears]
    vec = [(v.G.widened(), v.X.widened() if v.X is not None else None) for v in w.vectors]
    ref = O.dp_step(lin, w.ids, w.G_emb.widened(), w.V, w.C, lm=(w.lm.A.widened(), w.lm.G.widened()),
                    positions=True, vectors=vec)
    assert rel(ds.sq.cpu().numpy(), ref["sq"]).max() < TIGHT_BF16
    for k, want in ref["sums"].items():
        got = ds.outs[k].cpu().numpy()
        if k == "wpe":
            got = got[: w.T]
        assert frob_rel(got, want) < TOL_SUM, k
    # fused-noise step agrees with the unfused one on every tensor, vectors included
    a, b = P.upload(w), P.upload(w)
    P.dp_step(a, seed=3, step=1, fused=True)
    P.dp_step(b, seed=3, step=1, fused=False)
    torch.cuda.synchronize()
    for k in a.outs:
        assert torch.allclose(a.outs[k], b.outs[k], rtol=1e-5, atol=2e-6), k


# ------------------------------------------------------------- device-side failure path
def test_wait_limit_failure_path_leaves_context_usable():
    """Failure detection without a fault: with the barrier-wait limit set to zero every role of
    the TMA / tensor-core kernels gives up at its first unsatisfied wait, the kernels flag
    DP_DEV_TIMEOUT, let their copies in flight land, free their tensor memory and return.  The
    context stays usable and the same calls give correct results once the limit is restored."""
    L = dp.load()
    B, T, d, p, V = 4, 128, 256, 384, 1003
    A, G = host_linear(B, T, d, p, "bf16", seed=71)
    lin = dev_linear(A, G, dp.DP_NORM_GHOST)
    lin_direct = dev_linear(A, G, dp.DP_NORM_DIRECT)
    ids = torch.from_numpy(W.zipf_ids(B, T, V, 1.1, 72)).to(dev())
    G_emb, A_lm = P.to_device(W._normal((B, T, d), 1e-2, "bf16", 73)), P.to_device(W._normal((B, T, d), 1.0, "bf16", 74))
    G_lm = P.to_device(W._normal((B, T, V), 1e-2, "bf16", 75, ld=W.round_up(V, 8)))
    sq_in = torch.full((B,), 4.0, device=dev())

    def run_all():
        st = torch.zeros(1, dtype=torch.int32, device=dev())
        sq, sqd, cr = torch.zeros(B, device=dev()), torch.zeros(B, device=dev()), torch.zeros(B, device=dev())
        out = torch.zeros(p, d, device=dev())
        dp.dp_ghost_norms([lin], B, T, sq, dev_status=st)
        dp.dp_ghost_norms([lin_direct], B, T, sqd, dev_status=st)
        dp.dp_clip_accumulate(lin.A, lin.G, sq_in, 1.0, out, d=d, p=p, dev_status=st)
        dp.dp_tied_cross_term(ids, G_emb, A_lm, G_lm, V, cross=cr, d=d, dev_status=st)
        torch.cuda.synchronize()
        return int(st.item()), sq, sqd, out, cr

    good = run_all()
    assert good[0] == 0
    prev = L.dp_debug_set_wait_limit(0)
    try:
        bad = run_all()
    finally:
        L.dp_debug_set_wait_limit(prev)
    assert bad[0] & dp.DP_DEV_TIMEOUT
    again = run_all()
    assert again[0] == 0
    for a, b in zip(good[1:], again[1:]):
        assert torch.equal(a, b)
    want = O.linear_sq_norms(A.widened(), G.widened())
    assert rel(again[1].cpu().numpy(), want).max() < TIGHT_BF16


# ------------------------------------------------------------------ guard bands, edge sizes
def test_outputs_stay_inside_their_buffers():
    """Every output lives inside a larger allocation filled with a sentinel; after the calls only
    the output's own elements may have changed (a stand-in for a memory checker)."""
    B, T, d, p, V = 3, 100, 200, 300, 777
    A, G = host_linear(B, T, d, p, "bf16", seed=81, ldg=W.round_up(p, 8))     # TMA pitch, NaN padding
    lin = dev_linear(A, G)
    ids = torch.from_numpy(W.zipf_ids(B, T, V, 1.1, 82)).to(dev())
    G_emb = P.to_device(W._normal((B, T, d), 1e-2, "bf16", 83))
    pad, sent = 1024, -12345.0

    def guarded(n):
        buf = torch.full((n + 2 * pad,), sent, device=dev())
        return buf, buf[pad:pad + n]

    sq_buf, sq = guarded(B)
    sq.zero_()
    ldo = d + 8                                              # padded output pitch
    lin_buf, lin_out = guarded(p * ldo)
    emb_buf, emb_out = guarded(V * ldo)
    noise_buf, noise_out = guarded(4099)
    noise_out.zero_()
    dp.dp_ghost_norms([lin], B, T, sq)
    dp.dp_embed_norms(ids, G_emb, V, sq)
    dp.dp_clip_accumulate(lin.A, lin.G, sq, 1.0, lin_out.view(p, ldo)[:, :d], d=d, p=p)
    dp.dp_clip_accumulate_embed(ids, G_emb, V, sq, 1.0, emb_out.view(V, ldo)[:, :d])
    dp.dp_add_noise(noise_out, 1.0, 1.0, 1.0, 1, 2, 3)
    torch.cuda.synchronize()
    for buf in (sq_buf, lin_buf, emb_buf, noise_buf):
        assert bool((buf[:pad] == sent).all()) and bool((buf[-pad:] == sent).all())
    assert bool((lin_out.view(p, ldo)[:, d:] == sent).all())     # pitch padding untouched
    assert bool((emb_out.view(V, ldo)[:, d:] == sent).all())
    assert bool(torch.isfinite(lin_out.view(p, ldo)[:, :d]).all())


@pytest.mark.parametrize("B,T,d,p", [(1, 1024, 64, 72), (1, 640, 136, 64), (2, 129, 64, 64)])
def test_long_sequences_many_tile_pairs(B, T, d, p):
    """T well beyond one 128-row tile: 8 x 8 tile pairs, ragged last tile, both norm modes."""
    A, G = host_linear(B, T, d, p, "bf16", seed=T + d)
    want = O.linear_sq_norms(A.widened(), G.widened())
    for mode in (dp.DP_NORM_GHOST, dp.DP_NORM_DIRECT):
        sq = torch.zeros(B, device=dev())
        dp.dp_ghost_norms([dev_linear(A, G, mode)], B, T, sq)
        torch.cuda.synchronize()
        assert rel(sq.cpu().numpy(), want).max() < TIGHT_BF16, mode


def test_embedding_at_the_longest_supported_sequence():
    B, T, d, V = 1, 4096, 64, 50257
    ids = W.zipf_ids(B, T, V, 1.1, 91)
    G = W._normal((B, T, d), 1e-2, "bf16", 92)
    sq = torch.zeros(B, device=dev())
    fo = torch.zeros(B, T, dtype=torch.int32, device=dev())
    dp.dp_embed_norms(torch.from_numpy(ids).to(dev()), P.to_device(G), V, sq, first_occ=fo)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(fo.cpu().numpy(), O.first_occurrence(ids))
    assert rel(sq.cpu().numpy(), O.embed_sq_norms(ids, G.widened(), V)).max() < TIGHT_BF16
    with pytest.raises(dp.DpGhostError) as e:                # one token more is refused, not mis-run
        dp.dp_embed_norms(torch.zeros(1, 4097, dtype=torch.int32, device=dev()),
                          torch.zeros(1, 4097, d, dtype=torch.bfloat16, device=dev()), V, sq)
    assert e.value.status == 2


# ------------------------------------------------- slice noise, device step counter, step graph
def test_noise_on_slices_equals_the_whole_tensor_stream():
    seed, tid, step, n = 0x1234567890ABCDEF, 3, 9, 10007
    base = torch.randn(n, device=dev())
    whole = base.clone()
    dp.dp_add_noise(whole, 0.7, 1.3, 1.0, seed, tid, step)
    sliced = torch.empty_like(base)
    for lo, hi in [(0, 4096), (4096, 4100), (4100, 10007)]:
        part = base[lo:hi].clone()                         # its own 16-byte aligned buffer
        dp.dp_add_noise_slice(part, lo, 0.7, 1.3, 1.0, seed, tid, step)
        sliced[lo:hi] = part
        z = NO.standard_normals(hi - lo, seed, tid, step, start=lo)
        want = base[lo:hi].cpu().numpy().astype(np.float64) + 0.7 * 1.3 * z
        assert np.abs(part.cpu().numpy() - want).max() < 2e-6
    assert torch.equal(whole, sliced)                      # bit for bit the single-call result
    with pytest.raises(dp.DpGhostError):                   # a slice must start on a counter boundary
        dp.dp_add_noise_slice(base[:8].clone(), 2, 0.7, 1.3, 1.0, seed, tid, step)


def test_device_step_counter_is_added_to_the_step_word():
    seed, tid, n = 77, 1, 4099
    counter = torch.full((1,), 5, dtype=torch.int32, device=dev())
    x = torch.empty(n, device=dev())
    dp.dp_noise_step_device(counter)
    try:
        dp.dp_fill_noise(x, 1.0, 1.0, 1.0, seed, tid, 2)
        torch.cuda.synchronize()
    finally:
        dp.dp_noise_step_device(None)
    assert np.abs(x.cpu().numpy() - NO.standard_normals(n, seed, tid, 7)).max() < 1e-6
    dp.dp_fill_noise(x, 1.0, 1.0, 1.0, seed, tid, 2)       # cleared: the step is taken as given
    assert np.abs(x.cpu().numpy() - NO.standard_normals(n, seed, tid, 2)).max() < 1e-6


def test_step_graph_replays_equal_eager_steps():
    w = W.named_workload("cfg4", B=3, n_blocks=1, V=4099)
    a, b = P.upload(w), P.upload(w)
    g = P.StepGraph(a, seed=13, first_step=4)
    for k in range(3):                                     # replay k draws the noise of step 4 + k
        g.replay()
        P.dp_step(b, seed=13, step=4 + k)
        torch.cuda.synchronize()
        check_status(a.dev_status)
        for name in a.outs:
            assert torch.equal(a.outs[name], b.outs[name]), (k, name)
        assert torch.equal(a.sq, b.sq)
    assert int(g.counter.item()) == 7


@pytest.mark.parametrize("B,T,d,V,beta", [(3, 128, 768, 50257, 0.0), (5, 700, 100, 300, 1.0), (2, 40, 132, 7, 1.0)])
def test_sort_in_its_own_call_then_sorted_scatter(B, T, d, V, beta):
    """dp_embed_sort + dp_clip_accumulate_embed_sorted == dp_clip_accumulate_embed, bit for bit."""
    ids = W.zipf_ids(B, T, V, 1.1, 31)
    G = W._normal((B, T, d), 1e-2, "bf16", 32)
    sq_true = O.embed_sq_norms(ids, G.widened(), V)
    Cc = float(np.median(np.sqrt(sq_true)))
    sq = torch.from_numpy(sq_true.astype(np.float32)).to(dev())
    ids_d, G_d = torch.from_numpy(ids).to(dev()), P.to_device(G)
    out0 = torch.randn(V, d, device=dev())
    one, two = out0.clone(), out0.clone()
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_clip_accumulate_embed(ids_d, G_d, V, sq, Cc, one, beta=beta, dev_status=st)
    perm = torch.full((B * T,), -1, dtype=torch.int32, device=dev())
    seg = torch.full((V + 1,), -1, dtype=torch.int32, device=dev())
    dp.dp_embed_sort(ids_d, V, perm, seg, dev_status=st)
    dp.dp_clip_accumulate_embed_sorted(ids_d, G_d, V, sq, Cc, two, perm, seg, beta=beta, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    want_perm, want_seg = O.stable_token_sort(ids, V)
    np.testing.assert_array_equal(perm.cpu().numpy(), want_perm)
    np.testing.assert_array_equal(seg.cpu().numpy(), want_seg)
    assert torch.equal(one, two)
    _, R = O.clip_factors(sq.cpu().numpy().astype(np.float64), Cc)
    want = O.clipped_sum_embed(ids, G.widened(), R, V) + beta * out0.cpu().numpy().astype(np.float64)
    assert frob_rel(two.cpu().numpy(), want) < 1e-5


@pytest.mark.parametrize("B,T,d,p,ldg", [(2, 200, 192, 320, None), (1, 384, 128, 64, None), (3, 512, 256, 1024, None),
                                          (2, 300, 128, 5003, 5008), (2, 257, 72, 136, None)])
def test_pair_and_single_cta_gram_kernels_agree(B, T, d, p, ldg):
    """T > 128 runs on CTA pairs (256 x 256 Gram tiles); the single-CTA kernel (128 x 128 tiles)
    computes the same sum in another order.  Both against the oracle, and against each other."""
    A, G = host_linear(B, T, d, p, "bf16", seed=7 * T + p, ldg=ldg)
    want = O.linear_sq_norms(A.widened(), G.widened())
    got = {}
    for single in (False, True):
        prev = dp.dp_debug_ghost_single(single)
        try:
            sq = torch.zeros(B, device=dev())
            st = torch.zeros(1, dtype=torch.int32, device=dev())
            dp.dp_ghost_norms([dev_linear(A, G, dp.DP_NORM_GHOST)], B, T, sq, dev_status=st)
            torch.cuda.synchronize()
            check_status(st)
        finally:
            dp.dp_debug_ghost_single(prev)
        got[single] = sq.cpu().numpy()
        assert rel(got[single], want).max() < TIGHT_BF16, single
    assert rel(got[False], got[True]).max() < 1e-5


def test_pair_gram_kernel_wide_input_side_and_many_layers():
    """CTA-pair Gram kernel: the WIDE operand is the layer input (its columns are chunked across
    work items, each recomputing the narrow Gram), and more layers than one launch holds."""
    B, T = 2, 300
    # (a) d >> p: the split runs over A's columns
    rng = np.random.default_rng(5)
    A = W._normal((B, T, 5003), 1.0, "bf16", int(rng.integers(1 << 60)), ld=5008)
    G = W._normal((B, T, 128), 1e-2, "bf16", int(rng.integers(1 << 60)))
    sq = torch.zeros(B, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    dp.dp_ghost_norms([dev_linear(A, G, dp.DP_NORM_GHOST)], B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    assert rel(sq.cpu().numpy(), O.linear_sq_norms(A.widened(), G.widened())).max() < TIGHT_BF16
    # (b) 100 small layers: two launches of the pair kernel, one sum
    layers, want = [], np.zeros(B)
    for k in range(100):
        Ak, Gk = host_linear(B, T, 64, 72, "bf16", seed=1000 + k)
        layers.append(dev_linear(Ak, Gk, dp.DP_NORM_GHOST))
        want += O.linear_sq_norms(Ak.widened(), Gk.widened())
    sq = torch.zeros(B, device=dev())
    dp.dp_ghost_norms(layers, B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    assert rel(sq.cpu().numpy(), want).max() < TIGHT_BF16


def test_step_graph_with_positions_and_full_parameter_set():
    """Graph replays of a step that has a position table and every bias / LayerNorm parameter."""
    w = W.named_workload("cfg3", B=2, T=200, n_blocks=1, V=3001, full_model=True)
    a, b = P.upload(w), P.upload(w)
    g = P.StepGraph(a, seed=21, first_step=0)
    for k in range(2):
        g.replay()
        P.dp_step(b, seed=21, step=k)
        torch.cuda.synchronize()
        check_status(a.dev_status)
        for name in a.outs:
            assert torch.equal(a.outs[name], b.outs[name]), (k, name)


@pytest.mark.parametrize("cfg", ["cfg3", "cfg4"])
def test_bucketed_clip_phase_equals_the_plain_phases(cfg):
    """The multi-GPU step order on one GPU: clipped sums produced bucket by bucket (head first), each
    bucket handed to the exchange, which noises the slices it owns on its own stream -- same numbers
    as clip phase + noise phase issued in one piece (K may be split differently: 1e-5 Frobenius)."""
    from paper_2609_40335_b200 import parallel
    w = W.named_workload(cfg, B=3, T=100, n_blocks=2, V=3001)
    a, b = P.upload(w), P.upload(w)
    P.dp_step(a, seed=9, step=4, fused=False)
    P.norms_phase(b)
    ex = parallel.BucketedExchange(
        b.outs, lambda t, first, tid, st: dp.dp_add_noise_slice(t, first, b.sigma, b.C, 1.0, 9, tid, 4, stream=st))
    ex.begin_step()
    P.clip_phase_bucketed(b, ex, n_linear_buckets=3)
    ex.finish()
    torch.cuda.synchronize()
    check_status(b.dev_status)
    assert sorted(ex.submitted) == sorted(b.outs)
    for name in a.outs:
        assert frob_rel(b.outs[name].cpu().numpy(), a.outs[name].cpu().numpy()) < 1e-5, name
        lo, hi, mine = ex.owned[name]
        assert (lo, hi) == (0, a.outs[name].numel()) and mine.data_ptr() == b.outs[name].data_ptr()


@pytest.mark.parametrize("reserve", [16, 1000])
def test_reserved_sms_leave_the_results_unchanged(reserve):
    """dp_set_reserved_sms: the persistent kernels run on fewer SMs (what a data-parallel step sets
    so that its collectives find free SMs); every result still matches the oracle, with a second
    kernel holding SMs on another stream while the step runs."""
    prev = dp.dp_set_reserved_sms(reserve)
    try:
        assert prev == 0
        w = W.named_workload("cfg3", B=3, T=256, n_blocks=2, V=3001)
        ds = P.upload(w)
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            busy = torch.randn(4096, 4096, device=dev())
            for _ in range(4):
                busy = busy @ busy * 1e-2                   # keeps SMs busy beside the step
        P.dp_step(ds, noise=False)
        torch.cuda.synchronize()
        check_status(ds.dev_status)
        lin = [(l.A.widened(), l.G.widened()) for l in w.linears]
        ref = O.dp_step(lin, w.ids, w.G_emb.widened(), w.V, w.C, lm=(w.lm.A.widened(), w.lm.G.widened()),
                        tied=w.tied, positions=w.positions)
        assert rel(ds.sq.cpu().numpy(), ref["sq"]).max() < TIGHT_BF16
        for k, want in ref["sums"].items():
            got = ds.outs[k].cpu().numpy()
            if k == "wpe":
                got = got[: w.T]
            assert frob_rel(got, want) < TOL_SUM, k
    finally:
        back = dp.dp_set_reserved_sms(0)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert back == min(reserve, sms - 2)                    # clamped: at least one CTA pair stays


@pytest.mark.parametrize("cfg", ["cfg3", "cfg4"])
def test_repeated_steps_are_bitwise_identical(cfg):
    """Race check: the same step (same seed and step word) issued 40 times gives the same bits in
    every norm, clip factor and noised sum -- partial sums are combined in a fixed order everywhere,
    so any difference would be an unordered access."""
    w = W.named_workload(cfg, B=6, T=256 if cfg == "cfg3" else 128, n_blocks=2, V=5003)
    ds = P.upload(w)
    P.dp_step(ds, seed=5, step=7)
    torch.cuda.synchronize()
    ref = {k: v.clone() for k, v in ds.outs.items()}
    ref_sq, ref_clip = ds.sq.clone(), ds.clip.clone()
    for _ in range(40):
        P.dp_step(ds, seed=5, step=7)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    assert torch.equal(ds.sq, ref_sq) and torch.equal(ds.clip, ref_clip)
    for k in ref:
        assert torch.equal(ds.outs[k], ref[k]), k


# ------------------------------- full-size configurations in the launch configuration of the bench
def _oracle_example(w, i):
    """The oracle's squared norm (and, tied, cross term) of example i over every layer of w."""
    sl = slice(i, i + 1)
    lin = [(l.A.widened_rows(sl), l.G.widened_rows(sl)) for l in w.linears]
    return O.dp_step(lin, w.ids[sl], w.G_emb.widened_rows(sl), w.V, w.C,
                     lm=(w.lm.A.widened_rows(sl), w.lm.G.widened_rows(sl)), tied=w.tied,
                     positions=w.positions, want_sums=False)


def _full_size_graph_check(w, examples, layers, lm_rows, table_rows, seed=7, first_step=3):
    """One replay of the captured step graph (what bench.py times) at full size against the oracle:
    the norms (and cross terms) of `examples` (None: EVERY example of the batch), the clip factors of
    all, the noised clipped sums of `layers`, of rows `lm_rows` of the head and rows `table_rows` of
    the token table.  The clip factors that enter the expected sums are the ORACLE's wherever the
    oracle computed the example's norm, so a wrong norm on the device cannot cancel out."""
    ds = P.upload(w)
    g = P.StepGraph(ds, seed=seed, first_step=first_step)
    g.replay()
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    step = first_step                                        # replay k draws step first_step + k
    tid = P.tensor_ids(ds)
    sq_gpu = ds.sq.cpu().numpy().astype(np.float64)
    cross_gpu = ds.cross.cpu().numpy() if w.tied else None
    sq_ref = sq_gpu.copy()                                   # oracle values overwrite the checked entries
    for i in (range(w.B) if examples is None else examples):
        ref = _oracle_example(w, i)
        assert abs(sq_gpu[i] - ref["sq"][0]) / ref["sq"][0] < TIGHT_BF16, i
        sq_ref[i] = ref["sq"][0]
        if w.tied:
            scale = np.sqrt(ref["sq_in"][0] * ref["sq_out"][0])
            assert abs(cross_gpu[i] - ref["cross"][0]) / scale < TIGHT_BF16, i
    norms_ref, R = O.clip_factors(sq_ref, w.C)               # Eq. 7 on the oracle's norms
    assert rel(ds.clip.cpu().numpy(), R).max() < TIGHT_BF16
    assert rel(ds.norms.cpu().numpy(), norms_ref).max() < TIGHT_BF16
    _, R_own = O.clip_factors(sq_gpu, w.C)                   # the device's own Eq. 7 arithmetic
    assert rel(ds.clip.cpu().numpy(), R_own).max() < 1e-5
    amp = w.sigma * w.C

    def noise(name, n, start=0):
        return amp * NO.standard_normals(n, seed, tid[name], step, start=start)

    for k in layers:
        l = w.linears[k]
        want = O.clipped_sum_linear(l.A.widened(), l.G.widened(), R)
        want = want + noise(f"linear{k}", want.size).reshape(want.shape)
        assert frob_rel(ds.outs[f"linear{k}"].cpu().numpy(), want) < 5e-3, k
    # sampled rows of the head (its own matrix, or the shared table when tied)
    d = w.d_model
    head = "wte" if w.tied else "lm_head"
    rows = np.array(lm_rows)
    Gs = W.bf16_bits_to_f32(w.lm.G.data[:, :, rows]).astype(np.float64)
    want = O.clipped_sum_linear(w.lm.A.widened(), Gs, R)
    emb = O.clipped_sum_embed(w.ids, w.G_emb.widened(), R, w.V)
    if w.tied:
        want = want + emb[rows]                              # one table receives both (Eq. 8)
    for j, r_ in enumerate(rows):
        want[j] += noise(head, d, start=int(r_) * d)
    assert frob_rel(ds.outs[head].cpu().numpy()[rows], want) < 5e-3
    if not w.tied:
        trow = np.array(table_rows)
        want_t = emb[trow]
        for j, r_ in enumerate(trow):
            want_t[j] += noise("wte", d, start=int(r_) * d)
        assert frob_rel(ds.outs["wte"].cpu().numpy()[trow], want_t) < 5e-3
    if w.positions:
        pos_ids = np.tile(np.arange(w.T), (w.B, 1))
        want_p = O.clipped_sum_embed(pos_ids, w.G_emb.widened(), R, w.T)
        want_p = want_p + noise("wpe", want_p.size).reshape(want_p.shape)
        assert frob_rel(ds.outs["wpe"].cpu().numpy()[: w.T], want_p) < 5e-3


HEAD_ROWS = [0, 1, 255, 256, 25000, 50175, 50176, 50256]


def test_cfg2_full_size_graph_replay_sampled():
    w = W.named_workload("cfg2")
    hot = [int(np.bincount(w.ids.reshape(-1)).argmax()), int(w.ids[0, 0]), 0, 50256]
    # every example's norm against the oracle (about half a second of float64 each)
    _full_size_graph_check(w, examples=None, layers=(0, 23), lm_rows=HEAD_ROWS, table_rows=hot)


def test_cfg4_full_size_tied_graph_replay_sampled():
    w = W.named_workload("cfg4")
    hot = [int(np.bincount(w.ids.reshape(-1)).argmax())]
    # every example's tied norm and cross term against the oracle's materialised g_in + g_out
    _full_size_graph_check(w, examples=None, layers=(2, 47), lm_rows=HEAD_ROWS + hot, table_rows=[])


def test_cfg3_full_size_graph_replay_sampled():
    w = W.named_workload("cfg3")                             # B = 64, T = 256: the CTA-pair Gram kernel
    hot = [int(np.bincount(w.ids.reshape(-1)).argmax()), 50256]
    spread = (0, 9, 17, 26, 34, 45, 54, 63)                  # eight examples across the batch
    _full_size_graph_check(w, examples=spread, layers=(1,), lm_rows=HEAD_ROWS[:4], table_rows=hot)


def test_cfg5_cell_full_size_graph_replay_sampled():
    w = W.named_workload("cfg5", B=16, T=128)                # GPT-2-medium shape, 97 layers
    hot = [int(np.bincount(w.ids.reshape(-1)).argmax())]
    _full_size_graph_check(w, examples=(0, 7, 15), layers=(3, 95), lm_rows=HEAD_ROWS[:4], table_rows=hot)


def _host_rows(t, i, cols):
    """Example i of a device tensor (B, T, ld) as float64 on the host, padding columns dropped."""
    return t[i:i + 1, :, :cols].float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("B,T", [(16, 128), (64, 128), (256, 128), (16, 512), (64, 512), (256, 512)])
def test_cfg5_every_cell_one_example_against_the_oracle(B, T):
    """Each (B, T) cell of the GPT-2-medium sweep at full size (inputs drawn on the device, 97
    layers): one step, then the rows of a few examples are copied to the host and the float64
    oracle materialises their per-example gradients layer by layer -- norm, clip factor, and the
    device's whole vector of norms must be finite and deterministic."""
    ds = P.synthesize_on_device("cfg5", B, T, 1024, 24, seed=11)
    P.dp_step(ds, seed=5, step=2)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    sq = ds.sq.cpu().numpy().astype(np.float64)
    clip = ds.clip.cpu().numpy().astype(np.float64)
    assert np.isfinite(sq).all() and (sq > 0).all()
    every = ds.linears + [ds.lm]
    for i in sorted({0, B // 2 + 1, B - 1})[: (3 if T == 128 else 2)]:
        lin = [(_host_rows(l.A, i, l.d), _host_rows(l.G, i, l.p)) for l in ds.linears]
        ref = O.dp_step(lin, ds.ids[i:i + 1].cpu().numpy(), _host_rows(ds.G_emb, i, ds.d_model), ds.V,
                        ds.C, lm=(_host_rows(ds.lm.A, i, ds.lm.d), _host_rows(ds.lm.G, i, ds.lm.p)),
                        want_sums=False)
        assert abs(sq[i] - ref["sq"][0]) / ref["sq"][0] < TIGHT_BF16, (B, T, i)
        assert abs(clip[i] - ref["clip"][0]) / ref["clip"][0] < TIGHT_BF16, (B, T, i)
    assert len(every) == 97


@pytest.mark.parametrize("T", [256, 200])
def test_direct_norm_forced_on_every_gpt2_small_layer(T):
    """The per-layer switch at GPT-2-small shapes (config 3): DIRECT forced on all four block
    shapes and on the LM head (p = V), GHOST forced on the same layers, AUTO reported -- all three
    against the oracle's materialised per-example gradients."""
    B, V = 2, 50257
    shapes = [(768, 2304), (768, 768), (768, 3072), (3072, 768), (768, V)]
    host = [host_linear(B, T, d, p, "bf16", seed=31 * T + p + d, ldg=W.round_up(p, 8)) for d, p in shapes]
    want = [O.linear_sq_norms(A.widened(), G.widened()) for A, G in host]
    up = [(P.to_device(A), P.to_device(G)) for A, G in host]
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    for mode in (dp.DP_NORM_DIRECT, dp.DP_NORM_GHOST, dp.DP_NORM_AUTO):
        layers = [dp.Linear(a, g, d=d, p=p, mode=mode) for (a, g), (d, p) in zip(up, shapes)]
        # one call over all layers (the grouped launch) and one call per layer
        sq_all = torch.zeros(B, device=dev())
        used = dp.dp_ghost_norms(layers, B, T, sq_all, dev_status=st)
        torch.cuda.synchronize()
        check_status(st)
        if mode == dp.DP_NORM_AUTO:                          # T^2 <= d p everywhere: the rule picks GHOST
            assert used == [dp.DP_NORM_GHOST] * len(layers)
        else:
            assert used == [mode] * len(layers)
        assert rel(sq_all.cpu().numpy(), sum(want)).max() < TIGHT_BF16, mode
        for k, l in enumerate(layers):
            sq = torch.zeros(B, device=dev())
            dp.dp_ghost_norms([l], B, T, sq, dev_status=st)
            torch.cuda.synchronize()
            check_status(st)
            assert rel(sq.cpu().numpy(), want[k]).max() < TIGHT_BF16, (mode, shapes[k])


@pytest.mark.parametrize("B,T", [(64, 512), (256, 128), (256, 512)])
def test_cfg5_large_cells_against_library_gemms_on_the_device(B, T):
    """GPT-2-medium cells too large for the CPU oracle (inputs drawn on the device): sampled
    quantities are recomputed with plain library matrix products in float64 / fp32 on the GPU --
    the definition ||G_i^T A_i||_F^2 for sampled (example, layer) pairs, and sum_i R_i G_i^T A_i for a
    sampled layer -- and the whole step must be bitwise reproducible."""
    ds = P.synthesize_on_device("cfg5", B, T, 1024, 24, seed=3)
    P.dp_step(ds, seed=5, step=1)
    torch.cuda.synchronize()
    check_status(ds.dev_status)
    sq1 = ds.sq.clone()
    out1 = ds.outs["linear2"].clone()
    every = ds.linears + [ds.lm]
    # (a) per-example norm: all layers of one example, by definition, in float64 on the device
    i = B // 3
    want = 0.0
    for l in every:
        A = l.A[i, :, : l.d].double()
        G = l.G[i, :, : l.p].double()
        if l.p > 8192:                                       # the head: through the Gram identity's
            want += float(((A @ A.T) * (G @ G.T)).sum())     # T x T form (the p x d matrix is 0.4 GB)
        else:
            want += float((G.T @ A).pow(2).sum())
    ids = ds.ids[i].long()
    Ge = ds.G_emb[i, :, : ds.d_model].double()
    want += float(((ids[:, None] == ids[None, :]).double() * (Ge @ Ge.T)).sum())
    assert abs(float(sq1[i]) - want) / want < TIGHT_BF16
    # (b) clipped sum of one layer against a library GEMM with the rows scaled by R_i (fp32)
    R = torch.clamp(ds.C / ds.sq.sqrt(), max=1.0)
    l = ds.linears[2]
    Gs = (l.G[..., : l.p].float() * R[:, None, None]).reshape(-1, l.p)
    ref = Gs.T @ l.A[..., : l.d].float().reshape(-1, l.d)
    amp = ds.sigma * ds.C
    z = torch.zeros_like(ref)
    dp.dp_add_noise(z, ds.sigma, ds.C, 1.0, 5, P.tensor_ids(ds)["linear2"], 1)
    torch.cuda.synchronize()
    assert float((out1 - (ref + z)).norm() / (ref + z).norm()) < 5e-3
    assert amp > 0
    # (c) the step is deterministic
    P.dp_step(ds, seed=5, step=1)
    torch.cuda.synchronize()
    assert torch.equal(ds.sq, sq1) and torch.equal(ds.outs["linear2"], out1)


F32_TC_CASES = [(8, 128, 768, 3072), (3, 100, 72, 136), (2, 200, 192, 320), (2, 64, 3072, 768)]


@pytest.mark.parametrize("B,T,d,p", F32_TC_CASES)
@pytest.mark.parametrize("mode", [dp.DP_NORM_GHOST, dp.DP_NORM_DIRECT])
def test_fp32_inputs_on_tensor_cores_norms(B, T, d, p, mode):
    """DP_F32 layers that are large enough run on the bf16 tensor cores with every operand split
    into two bf16 terms (three products per product).  Norms against the oracle at the fp32
    tolerance 1e-4, and against the plain fp32 FMA kernels (the cross-check path)."""
    A, G = host_linear(B, T, d, p, "f32", seed=17 * T + d + p)
    lin = dev_linear(A, G, mode)
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    sq = torch.zeros(B, device=dev())
    assert dp.dp_ghost_norms_ws_bytes([lin], B, T) > 0                 # the split path is the one taken
    used = dp.dp_ghost_norms([lin], B, T, sq, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    assert used == [mode]
    want = O.linear_sq_norms(A.widened(), G.widened())
    assert rel(sq.cpu().numpy(), want).max() < TOL_F32
    assert rel(sq.cpu().numpy(), want).max() < 2e-5                    # what two bf16 terms give
    prev = dp.dp_debug_force_fma(1)
    try:
        sq_fma = torch.zeros(B, device=dev())
        dp.dp_ghost_norms([lin], B, T, sq_fma, dev_status=st)
        torch.cuda.synchronize()
    finally:
        dp.dp_debug_force_fma(prev)
    assert rel(sq.cpu().numpy(), sq_fma.cpu().numpy()).max() < 5e-5


@pytest.mark.parametrize("B,T,d,p", F32_TC_CASES)
@pytest.mark.parametrize("beta", [0.0, 1.0])
def test_fp32_inputs_on_tensor_cores_clipped_sums(B, T, d, p, beta):
    """Clipped sum of a DP_F32 layer on the tensor cores: R_i multiplies G in fp32 before the split,
    so the result keeps fp32-class accuracy (1e-4 Frobenius asserted; bf16 inputs get 5e-3)."""
    A, G = host_linear(B, T, d, p, "f32", seed=5 * T + d + p)
    lin = dev_linear(A, G)
    rng = np.random.default_rng(B + T)
    sq = torch.from_numpy(rng.uniform(0.25, 9.0, B).astype(np.float32)).to(dev())   # both branches of min
    Cc = 1.5
    _, R = O.clip_factors(sq.cpu().numpy().astype(np.float64), Cc)
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    init = torch.from_numpy(rng.standard_normal((p, d)).astype(np.float32)).to(dev())
    out = init.clone()
    dp.dp_clip_accumulate_grouped([lin], B, T, sq, Cc, [out], beta=beta, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    want = O.clipped_sum_linear(A.widened(), G.widened(), R) + beta * init.cpu().numpy().astype(np.float64)
    assert frob_rel(out.cpu().numpy(), want) < 1e-4
    # fused noise equals clipped sum + stand-alone noise, bit for bit
    a, b = init.clone(), init.clone()
    dp.dp_clip_accumulate_noise_grouped([lin], B, T, sq, Cc, [a], 0.7, 1.0, 5, [3], 9, beta=beta, dev_status=st)
    dp.dp_clip_accumulate_grouped([lin], B, T, sq, Cc, [b], beta=beta, dev_status=st)
    dp.dp_add_noise(b, 0.7, Cc, 1.0, 5, 3, 9)
    torch.cuda.synchronize()
    check_status(st)
    assert torch.equal(a, b)


def test_tensor_maps_are_encoded_once_per_tensor():
    """Calls issued one by one (no CUDA graph) reuse the TMA tensor maps of tensors they have seen:
    the second identical call makes no driver encode at all."""
    B, T = 2, 128
    layers = [dev_linear(*host_linear(B, T, 128, 256, "bf16", seed=k)) for k in range(3)]
    sq = torch.zeros(B, device=dev())
    outs = [torch.empty(256, 128, device=dev()) for _ in layers]
    L = dp.load()

    def one_step():
        dp.dp_ghost_norms(layers, B, T, sq)
        dp.dp_clip_accumulate_grouped(layers, B, T, sq, 1.0, outs)
    one_step()
    n0 = L.dp_debug_tensor_map_encodes()
    one_step()
    one_step()
    torch.cuda.synchronize()
    assert L.dp_debug_tensor_map_encodes() == n0
    other = dev_linear(*host_linear(B, T, 128, 256, "bf16", seed=99))
    dp.dp_ghost_norms([other], B, T, sq)
    assert L.dp_debug_tensor_map_encodes() == n0 + 2          # a new tensor pair: two new maps


def test_bad_squared_norms_fail_closed():
    """Eq. 7 on corrupted norms: NaN / inf give a factor of 0 (the example leaves the sum, it is
    never added unclipped); a tiny negative value (rounding of in + out + 2 cross) counts as 0."""
    sq = torch.tensor([float("nan"), float("inf"), -1e-9, 0.0, 4.0, 0.25, -float("inf")], device=dev())
    clip, norms = torch.empty_like(sq), torch.empty_like(sq)
    dp.dp_clip_factors(sq, 1.0, clip=clip, norms=norms)
    torch.cuda.synchronize()
    assert clip.cpu().tolist() == [0.0, 0.0, 1.0, 1.0, 0.5, 1.0, 0.0]
    # and inside a clipped sum: the NaN example contributes nothing
    B, T, d, p = 3, 64, 64, 128
    A, G = host_linear(B, T, d, p, "bf16", seed=77)
    lin = dev_linear(A, G)
    sq3 = torch.tensor([4.0, float("nan"), 1e-12], device=dev())
    out = torch.empty(p, d, device=dev())
    dp.dp_clip_accumulate_grouped([lin], B, T, sq3, 1.0, [out])
    torch.cuda.synchronize()
    want = O.clipped_sum_linear(A.widened(), G.widened(), np.array([0.5, 0.0, 1.0]))
    assert np.isfinite(out.cpu().numpy()).all()
    assert frob_rel(out.cpu().numpy(), want) < 5e-3


def test_fused_noise_on_outputs_that_are_only_4_byte_aligned():
    """The fused entry points accept any fp32 output tensor: a base that is 4-byte but not 16-byte
    aligned takes the scalar branch of the noise pass (same values as the aligned call, no fault)."""
    B, T, d, V = 4, 64, 64, 301
    ids = torch.from_numpy(W.zipf_ids(B, T, V, 1.1, 3)).to(dev())
    Ge = P.to_device(W._normal((B, T, d), 1e-2, "bf16", 4))
    sq = torch.full((B,), 9.0, device=dev())
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    aligned = torch.empty(V, d, device=dev())
    buf = torch.empty(V * d + 8, device=dev())
    odd = buf[1:1 + V * d].view(V, d)                       # data_ptr() % 16 == 4
    assert odd.data_ptr() % 16 == 4
    for out in (aligned, odd):
        dp.dp_clip_accumulate_embed_noise(ids, Ge, V, sq, 1.0, out, 0.7, 1.0, 5, 2, 9, beta=0.0,
                                          dev_status=st)
    # fp32 linear layer with fused noise: the unfused path adds noise with the same kernel
    A, G = host_linear(B, T, d, 96, "f32", seed=8)
    lin = dev_linear(A, G)
    o1 = torch.empty(96, d, device=dev())
    buf2 = torch.empty(96 * d + 8, device=dev())
    o2 = buf2[1:1 + 96 * d].view(96, d)
    for out in (o1, o2):
        dp.dp_clip_accumulate_noise_grouped([lin], B, T, sq, 1.0, [out], 0.7, 1.0, 5, [3], 9, dev_status=st)
    torch.cuda.synchronize()
    check_status(st)
    assert torch.equal(aligned, odd) and torch.equal(o1, o2)


def test_precomputed_clip_factors_and_fused_accumulator_join():
    """sq = None makes `clip` an input of the clip-accumulate calls; dp_clip_factors_sum joins two
    norm accumulators and takes Eq. 7 in one kernel.  Both must equal the plain calls bit for bit."""
    B, T, d, p, V = 5, 100, 136, 264, 777
    A, G = host_linear(B, T, d, p, "bf16", seed=3, ldg=W.round_up(p, 8))
    lin = dev_linear(A, G)
    rng = np.random.default_rng(4)
    sq_a = torch.from_numpy(rng.uniform(0.1, 3.0, B).astype(np.float32)).to(dev())
    sq_b = torch.from_numpy(rng.uniform(0.1, 3.0, B).astype(np.float32)).to(dev())
    # (a) the fused join
    want_sq = sq_a + sq_b
    clip_ref, norms_ref = torch.empty(B, device=dev()), torch.empty(B, device=dev())
    dp.dp_clip_factors(want_sq, 1.0, clip=clip_ref, norms=norms_ref)
    sq, clip, norms = sq_a.clone(), torch.empty(B, device=dev()), torch.empty(B, device=dev())
    dp.dp_clip_factors_sum(sq, sq_b, 1.0, clip=clip, norms=norms)
    torch.cuda.synchronize()
    assert torch.equal(sq, want_sq) and torch.equal(clip, clip_ref) and torch.equal(norms, norms_ref)
    _, R = O.clip_factors(want_sq.cpu().numpy().astype(np.float64), 1.0)
    assert rel(clip.cpu().numpy(), R).max() < 1e-6
    # (b) factors given instead of squared norms: linear layer, embedding, vector parameter
    one, two = torch.empty(p, d, device=dev()), torch.empty(p, d, device=dev())
    dp.dp_clip_accumulate_grouped([lin], B, T, want_sq, 1.0, [one])
    dp.dp_clip_accumulate_grouped([lin], B, T, None, 1.0, [two], clip=clip)
    ids = torch.from_numpy(W.zipf_ids(B, T, V, 1.1, 5)).to(dev())
    Ge = P.to_device(W._normal((B, T, d), 1e-2, "bf16", 6))
    e1, e2 = torch.empty(V, d, device=dev()), torch.empty(V, d, device=dev())
    dp.dp_clip_accumulate_embed(ids, Ge, V, want_sq, 1.0, e1)
    dp.dp_clip_accumulate_embed(ids, Ge, V, None, 1.0, e2, clip=clip)
    vec = [dp.Vector(lin.G, None, p=p)]
    v1, v2 = torch.empty(p, device=dev()), torch.empty(p, device=dev())
    dp.dp_clip_accumulate_vectors(vec, B, T, want_sq, 1.0, [v1])
    dp.dp_clip_accumulate_vectors(vec, B, T, None, 1.0, [v2], clip=clip)
    torch.cuda.synchronize()
    assert torch.equal(one, two) and torch.equal(e1, e2) and torch.equal(v1, v2)
    with pytest.raises(dp.DpGhostError):                 # neither squared norms nor factors
        dp.dp_clip_accumulate_grouped([lin], B, T, None, 1.0, [two])
