"""Pins for oracle/dp_oracle.py against things other than itself:
per-example autograd on tiny float64 models, the Gram identity, closed forms,
Eq. 11 on materialised matrices, library GEMM / argsort, brute-force loops.
"""
import os

import numpy as np
import pytest
import torch

from oracle import dp_oracle as O

RNG = np.random.default_rng(1234)


# --------------------------------------------------------------- tiny autograd model
class Tiny(torch.nn.Module):
    """wte (+wpe) -> linear1 -> tanh -> linear2 -> head, all without biases."""

    def __init__(self, V, d, h, T, tied, positions):
        super().__init__()
        g = torch.Generator().manual_seed(7)
        mk = lambda *s: torch.nn.Parameter(torch.randn(*s, generator=g, dtype=torch.float64) * 0.5)
        self.wte = mk(V, d)
        self.wpe = mk(T, d) if positions else None
        self.w1 = mk(h, d)
        self.w2 = mk(d, h)
        self.head = None if tied else mk(V, d)
        self.tied = tied

    def forward(self, ids, keep):
        B, T = ids.shape
        h0 = self.wte[ids]
        if self.wpe is not None:
            h0 = h0 + self.wpe[torch.arange(T)][None]
        keep["h0"] = h0
        z1 = h0 @ self.w1.T
        keep["z1"] = z1
        a1 = torch.tanh(z1)
        keep["a1"] = a1
        z2 = a1 @ self.w2.T
        keep["z2"] = z2
        hf = z2 + h0
        keep["hf"] = hf
        Wout = self.wte if self.tied else self.head
        logits = hf @ Wout.T
        keep["logits"] = logits
        return logits


def _per_example_losses(model, ids, labels, keep):
    logits = model(ids, keep)
    B, T, V = logits.shape
    ls = torch.nn.functional.cross_entropy(logits.reshape(B * T, V), labels.reshape(-1),
                                           reduction="none").reshape(B, T)
    return ls.sum(dim=1)


@pytest.mark.parametrize("tied,positions", [(False, False), (False, True), (True, False), (True, True)])
def test_oracle_matches_per_example_autograd(tied, positions):
    V, d, h, T, B = 11, 6, 5, 7, 4
    model = Tiny(V, d, h, T, tied, positions)
    g = torch.Generator().manual_seed(3)
    ids = torch.randint(0, V, (B, T), generator=g)
    ids[0, 3] = ids[0, 1]            # force a repeated token
    ids[1, :] = ids[1, 0]            # one example with a single token id
    labels = torch.randint(0, V, (B, T), generator=g)
    params = [p for p in model.parameters()]
    names = [n for n, _ in model.named_parameters()]

    # brute force: one autograd call per example
    per_ex = []
    for i in range(B):
        keep = {}
        li = _per_example_losses(model, ids[i:i + 1], labels[i:i + 1], keep)[0]
        per_ex.append(torch.autograd.grad(li, params))
    sq_true = np.array([sum(float((g_ ** 2).sum()) for g_ in gs) for gs in per_ex])

    # batch pass with hooks: layer inputs A and output gradients G
    keep = {}
    total = _per_example_losses(model, ids, labels, keep).sum()
    outs = [keep["h0"], keep["z1"], keep["z2"], keep["logits"]]
    G_h0, G_z1, G_z2, G_log = torch.autograd.grad(total, outs)
    A1, A2, A_lm = keep["h0"].detach().numpy(), keep["a1"].detach().numpy(), keep["hf"].detach().numpy()
    linears = [(A1, G_z1.numpy()), (A2, G_z2.numpy())]
    Cclip = float(np.median(np.sqrt(sq_true)))   # some examples clipped, some not
    res = O.dp_step(linears, ids.numpy(), G_h0.numpy(), V, Cclip,
                    lm=(A_lm, G_log.numpy()), tied=tied, positions=positions)
    np.testing.assert_allclose(res["sq"], sq_true, rtol=1e-10)
    assert (res["clip"] < 1).any() and (res["clip"] == 1).any()

    # clipped sums against sum_i R_i * autograd gradient
    R = np.minimum(1.0, Cclip / np.sqrt(sq_true))
    want = {n: sum(R[i] * per_ex[i][k].numpy() for i in range(B)) for k, n in enumerate(names)}
    got = res["sums"]
    np.testing.assert_allclose(got["linear0"], want["w1"], rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(got["linear1"], want["w2"], rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(got["wte"], want["wte"], rtol=1e-9, atol=1e-12)
    if positions:
        np.testing.assert_allclose(got["wpe"], want["wpe"], rtol=1e-9, atol=1e-12)
    if not tied:
        np.testing.assert_allclose(got["lm_head"], want["head"], rtol=1e-9, atol=1e-12)
    else:
        assert "lm_head" not in got


# ------------------------------------------------------------------ linear-layer pins
def test_gram_identity():
    B, T, d, p = 3, 9, 5, 4
    A, G = RNG.standard_normal((B, T, d)), RNG.standard_normal((B, T, p))
    want = np.array([np.sum((A[i] @ A[i].T) * (G[i] @ G[i].T)) for i in range(B)])
    np.testing.assert_allclose(O.linear_sq_norms(A, G), want, rtol=1e-12)


def test_eq5_single_token_closed_form():
    B, d, p = 5, 7, 3
    A, G = RNG.standard_normal((B, 1, d)), RNG.standard_normal((B, 1, p))
    want = (A[:, 0] ** 2).sum(1) * (G[:, 0] ** 2).sum(1)
    np.testing.assert_allclose(O.linear_sq_norms(A, G), want, rtol=1e-12)


def test_orthonormal_activations_reduce_to_token_norms():
    T, d, p = 6, 8, 5
    Q, _ = np.linalg.qr(RNG.standard_normal((d, d)))
    A = Q[:T][None]                       # orthonormal rows
    G = RNG.standard_normal((1, T, p))
    np.testing.assert_allclose(O.linear_sq_norms(A, G), [(G ** 2).sum()], rtol=1e-12)


def test_scaling_and_token_permutation():
    B, T, d, p = 2, 8, 4, 6
    A, G = RNG.standard_normal((B, T, d)), RNG.standard_normal((B, T, p))
    base = O.linear_sq_norms(A, G)
    np.testing.assert_allclose(O.linear_sq_norms(A, -3.0 * G), 9.0 * base, rtol=1e-12)
    perm = RNG.permutation(T)
    np.testing.assert_allclose(O.linear_sq_norms(A[:, perm], G[:, perm]), base, rtol=1e-12)
    # a transposed operand must change the answer (guards against G A^T style slips)
    assert O.linear_example_grad(A[0], G[0]).shape == (p, d)


def test_linear_grad_entry_by_entry():
    T, d, p = 3, 2, 2
    A, G = RNG.standard_normal((T, d)), RNG.standard_normal((T, p))
    P = O.linear_example_grad(A, G)
    for r in range(p):
        for c in range(d):
            assert P[r, c] == pytest.approx(sum(G[t, r] * A[t, c] for t in range(T)), rel=1e-12)


# ------------------------------------------------------------------ embedding pins
def test_embedding_distinct_and_equal_ids():
    T, d, V = 6, 4, 20
    G = RNG.standard_normal((2, T, d))
    ids = np.stack([RNG.permutation(V)[:T], np.full(T, 5)])
    got = O.embed_sq_norms(ids, G, V)
    assert got[0] == pytest.approx((G[0] ** 2).sum(), rel=1e-12)
    assert got[1] == pytest.approx((G[1].sum(0) ** 2).sum(), rel=1e-12)


def test_embedding_pairs_bruteforce_and_onehot_linear():
    B, T, d, V = 3, 8, 5, 6
    ids = RNG.integers(0, V, (B, T))
    G = RNG.standard_normal((B, T, d))
    want = np.zeros(B)
    for i in range(B):
        for t in range(T):
            for s in range(T):
                if ids[i, t] == ids[i, s]:
                    want[i] += G[i, t] @ G[i, s]
    np.testing.assert_allclose(O.embed_sq_norms(ids, G, V), want, rtol=1e-12)
    onehot = np.eye(V)[ids]                               # (B, T, V): the layer's input
    # embedding = linear layer with one-hot input; weight gradient is (d, V) there
    np.testing.assert_allclose(O.linear_sq_norms(onehot, G), want, rtol=1e-12)
    np.testing.assert_allclose(O.embed_example_grad(ids[0], G[0], V),
                               O.linear_example_grad(onehot[0], G[0]).T, rtol=1e-12)


# ------------------------------------------------------------------------ tied pins
def test_tied_identity_eq11_and_cauchy_schwarz():
    B, T, d, V = 3, 7, 4, 9
    ids = RNG.integers(0, V, (B, T))
    G_emb, A_lm, G_lm = (RNG.standard_normal((B, T, d)), RNG.standard_normal((B, T, d)),
                         RNG.standard_normal((B, T, V)))
    r = O.tied_sq_norms(ids, G_emb, A_lm, G_lm, V)
    np.testing.assert_allclose(r["tied"], r["in"] + r["out"] + 2 * r["cross"], rtol=1e-12)
    assert (np.abs(r["cross"]) <= np.sqrt(r["in"] * r["out"]) * (1 + 1e-12)).all()
    np.testing.assert_allclose(r["in"], O.embed_sq_norms(ids, G_emb, V), rtol=1e-12)
    np.testing.assert_allclose(r["out"], O.linear_sq_norms(A_lm, G_lm), rtol=1e-12)
    # independent expansion of the inner product over token pairs
    want = np.zeros(B)
    for i in range(B):
        for t in range(T):
            for s in range(T):
                want[i] += G_lm[i, s, ids[i, t]] * (G_emb[i, t] @ A_lm[i, s])
    np.testing.assert_allclose(r["cross"], want, rtol=1e-10)
    assert np.abs(r["cross"]).min() > 1e-6     # the term is really there (Eq. 12)


# ------------------------------------------------------------------------ clip pins
def test_clip_factor_properties():
    sq = np.array([0.0, 0.25, 1.0, 4.0, 1e-30, 1e30])
    norms, R = O.clip_factors(sq, 1.0)
    np.testing.assert_allclose(norms, [0, 0.5, 1, 2, 1e-15, 1e15])
    np.testing.assert_allclose(R, [1, 1, 1, 0.5, 1, 1e-15])
    assert ((R > 0) & (R <= 1)).all()
    assert (R * norms <= 1.0 * (1 + 1e-12)).all()
    _, R2 = O.clip_factors(sq, 0.05)
    np.testing.assert_allclose(R2[3], 0.025)


# ------------------------------------------------------------------- aggregate pins
def test_unclipped_sum_is_one_library_gemm():
    B, T, d, p = 4, 6, 5, 3
    A, G = RNG.standard_normal((B, T, d)), RNG.standard_normal((B, T, p))
    got = O.clipped_sum_linear(A, G, np.ones(B))
    want = G.reshape(B * T, p).T @ A.reshape(B * T, d)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)


def test_clipped_sum_weights_and_norm_bound():
    B, T, d, p, C = 5, 4, 6, 3, 0.7
    A, G = RNG.standard_normal((B, T, d)), RNG.standard_normal((B, T, p))
    _, R = O.clip_factors(O.linear_sq_norms(A, G), C)
    S = O.clipped_sum_linear(A, G, R)
    assert np.linalg.norm(S) <= B * C * (1 + 1e-12)
    one = O.clipped_sum_linear(A[:1], G[:1], R[:1])
    np.testing.assert_allclose(one, R[0] * (G[0].T @ A[0]), rtol=1e-12)
    assert np.linalg.norm(one) == pytest.approx(min(C, np.linalg.norm(G[0].T @ A[0])), rel=1e-12)


def test_clipped_sum_embed_rows():
    B, T, d, V = 3, 5, 4, 7
    ids = RNG.integers(0, V, (B, T))
    G = RNG.standard_normal((B, T, d))
    R = np.array([0.5, 1.0, 0.25])
    S = O.clipped_sum_embed(ids, G, R, V)
    want = np.zeros((V, d))
    np.add.at(want, ids.reshape(-1), (R[:, None, None] * G).reshape(-1, d))
    np.testing.assert_allclose(S, want, rtol=1e-12, atol=1e-14)
    untouched = sorted(set(range(V)) - set(ids.reshape(-1).tolist()))
    assert (S[untouched] == 0).all()


# --------------------------------------------------------------------- integer pins
def test_integer_side_outputs():
    B, T, V = 4, 33, 9
    ids = RNG.integers(0, V, (B, T)).astype(np.int32)
    first = O.first_occurrence(ids)
    for i in range(B):
        for t in range(T):
            assert first[i, t] == list(ids[i]).index(ids[i, t])
    perm, seg = O.stable_token_sort(ids, V)
    np.testing.assert_array_equal(perm, np.argsort(ids.reshape(-1), kind="stable"))
    np.testing.assert_array_equal(seg, np.concatenate([[0], np.cumsum(np.bincount(ids.reshape(-1), minlength=V))]))


# -------------------------------------------------------- additivity (Eq. 6 / Eq. 10)
def test_untied_blocks_add_and_tied_blocks_do_not():
    B, T, d, V = 2, 5, 4, 6
    ids = RNG.integers(0, V, (B, T))
    G_emb, A_lm, G_lm = (RNG.standard_normal((B, T, d)), RNG.standard_normal((B, T, d)),
                         RNG.standard_normal((B, T, V)))
    lin = [(RNG.standard_normal((B, T, d)), RNG.standard_normal((B, T, 3)))]
    u = O.dp_step(lin, ids, G_emb, V, 1.0, lm=(A_lm, G_lm), tied=False, want_sums=False)
    t = O.dp_step(lin, ids, G_emb, V, 1.0, lm=(A_lm, G_lm), tied=True, want_sums=False)
    parts = O.linear_sq_norms(*lin[0]) + O.embed_sq_norms(ids, G_emb, V) + O.linear_sq_norms(A_lm, G_lm)
    np.testing.assert_allclose(u["sq"], parts, rtol=1e-12)
    np.testing.assert_allclose(t["sq"] - u["sq"], 2 * t["cross"], rtol=1e-9)
    assert np.abs(t["sq"] - u["sq"]).min() > 1e-6


# --------------------------------------------- shapes pinned by the paper's Table 1
def test_workload_shapes_reproduce_table1_counts():
    from paper_2609_40335_b200.workloads import GPT2_VOCAB, gpt2_block_shapes
    path = os.path.join(os.path.dirname(__file__), "golden", "table1_param_counts.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    d = 768
    for model, tied, count in rows:
        blocks = 6 if model == "distilgpt2" else 12
        per_block = sum(dd * pp + pp for dd, pp in gpt2_block_shapes(d)) + 2 * 2 * d
        n = GPT2_VOCAB * d + 1024 * d + blocks * per_block + 2 * d
        if tied == "0":
            n += GPT2_VOCAB * d
        assert n == int(count), (model, tied)


# ------------------------------------------- vector parameters: biases and LayerNorm
class TinyFull(torch.nn.Module):
    """wte -> LayerNorm -> linear1 (+bias) -> tanh -> linear2 (+bias) -> untied head (no bias)."""

    def __init__(self, V, d, h):
        super().__init__()
        g = torch.Generator().manual_seed(11)
        mk = lambda *s: torch.nn.Parameter(torch.randn(*s, generator=g, dtype=torch.float64) * 0.5)
        self.wte, self.gamma, self.beta = mk(V, d), mk(d), mk(d)
        self.w1, self.b1, self.w2, self.b2, self.head = mk(h, d), mk(h), mk(d, h), mk(d), mk(V, d)

    def forward(self, ids, keep):
        h0 = self.wte[ids]
        keep["h0"] = h0
        mu = h0.mean(-1, keepdim=True)
        var = ((h0 - mu) ** 2).mean(-1, keepdim=True)
        xhat = (h0 - mu) / torch.sqrt(var + 1e-5)
        keep["xhat"] = xhat
        y = self.gamma * xhat + self.beta
        keep["y"] = y
        z1 = y @ self.w1.T + self.b1
        keep["z1"] = z1
        a1 = torch.tanh(z1)
        keep["a1"] = a1
        z2 = a1 @ self.w2.T + self.b2
        keep["z2"] = z2
        logits = z2 @ self.head.T
        keep["logits"] = logits
        return logits


def test_oracle_vector_parameters_match_per_example_autograd():
    V, d, h, T, B = 9, 6, 5, 7, 4
    model = TinyFull(V, d, h)
    g = torch.Generator().manual_seed(4)
    ids = torch.randint(0, V, (B, T), generator=g)
    labels = torch.randint(0, V, (B, T), generator=g)
    params = list(model.parameters())
    names = [n for n, _ in model.named_parameters()]

    def losses(idx, keep):
        logits = model(ids[idx], keep)
        n = logits.shape[0]
        return torch.nn.functional.cross_entropy(logits.reshape(n * T, V), labels[idx].reshape(-1),
                                                 reduction="none").reshape(n, T).sum(1)

    per_ex = [torch.autograd.grad(losses(slice(i, i + 1), {})[0], params) for i in range(B)]
    sq_true = np.array([sum(float((x ** 2).sum()) for x in gs) for gs in per_ex])
    keep = {}
    total = losses(slice(0, B), keep).sum()
    G_h0, G_y, G_z1, G_z2, G_log = torch.autograd.grad(
        total, [keep["h0"], keep["y"], keep["z1"], keep["z2"], keep["logits"]])
    npy = lambda t: t.detach().numpy()
    linears = [(npy(keep["y"]), npy(G_z1)), (npy(keep["a1"]), npy(G_z2))]
    vectors = [(npy(G_y), npy(keep["xhat"])), (npy(G_y), None), (npy(G_z1), None), (npy(G_z2), None)]
    Cc = float(np.median(np.sqrt(sq_true)))
    res = O.dp_step(linears, ids.numpy(), npy(G_h0), V, Cc, lm=(npy(keep["z2"]), npy(G_log)),
                    vectors=vectors)
    np.testing.assert_allclose(res["sq"], sq_true, rtol=1e-10)
    R = np.minimum(1.0, Cc / np.sqrt(sq_true))
    want = {n: sum(R[i] * per_ex[i][k].numpy() for i in range(B)) for k, n in enumerate(names)}
    for key, name in [("vector0", "gamma"), ("vector1", "beta"), ("vector2", "b1"), ("vector3", "b2"),
                      ("linear0", "w1"), ("linear1", "w2"), ("lm_head", "head"), ("wte", "wte")]:
        np.testing.assert_allclose(res["sums"][key], want[name], rtol=1e-9, atol=1e-12)


def test_vector_gradient_special_cases():
    B, T, p = 3, 5, 4
    G, X = RNG.standard_normal((B, T, p)), RNG.standard_normal((B, T, p))
    np.testing.assert_allclose(O.vector_sq_norms(G), (G.sum(1) ** 2).sum(1), rtol=1e-12)
    np.testing.assert_allclose(O.vector_sq_norms(G, X), ((G * X).sum(1) ** 2).sum(1), rtol=1e-12)
    np.testing.assert_allclose(O.vector_sq_norms(G, np.ones_like(G)), O.vector_sq_norms(G), rtol=1e-12)
    # a bias is a linear layer whose input is the constant 1 (Eq. 4 with a_t = 1)
    ones = np.ones((B, T, 1))
    np.testing.assert_allclose(O.vector_sq_norms(G), O.linear_sq_norms(ones, G), rtol=1e-12)
    R = np.array([0.5, 1.0, 0.25])
    np.testing.assert_allclose(O.clipped_sum_vector(G, X, R), np.einsum("i,itp,itp->p", R, G, X), rtol=1e-12)
    np.testing.assert_allclose(O.clipped_sum_vector(G, None, R),
                               O.clipped_sum_linear(ones, G, R)[:, 0], rtol=1e-12)
