"""Plain float64 CPU oracle of the DP-SGD step with per-example clipping.

TEST INFRASTRUCTURE ONLY: slow on purpose, never imported by the product
package, shares no code with the CUDA path.

The clipped, noised gradient sum of DP-SGD is an exact quantity (Eq. 2, Eq. 3),
so this file is the plain definition: every per-example gradient is
materialised, its Frobenius norm is taken, the clip coefficient of Eq. 7 is
applied and the clipped gradients are summed.  Nothing here uses the ghost
(Gram) identity, token-equality tricks or any blocking: that is what the CUDA
path does and what the tests compare against this file.

Notation (paper, Sec. II): for a linear layer, sample i has activations
a_{i,t} (rows of A_i, T x d) and back-propagated signals delta_{i,t} (rows of
G_i, T x p).  Eq. 4 gives the per-token gradient delta a^T; a sequence sums
them: g_i = sum_t delta_{i,t} a_{i,t}^T = G_i^T A_i  (p x d, the layout of a
linear layer's weight).

Pins (tests/test_oracle_*.py): per-example autograd on tiny float64 models
(tied and untied), the Gram identity sum_{t,s}(a_t.a_s)(g_t.g_s), the T=1
closed form of Eq. 5, Eq. 11 on materialised matrices, all-ones clip factors
reducing to one library GEMM, brute-force loops for the integer outputs.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "linear_example_grad", "linear_sq_norms", "embed_example_grad", "embed_sq_norms",
    "tied_sq_norms", "clip_factors", "clipped_sum_linear", "clipped_sum_embed",
    "vector_example_grad", "vector_sq_norms", "clipped_sum_vector",
    "first_occurrence", "stable_token_sort", "dp_step",
]


def _f64(x):
    return np.asarray(x, dtype=np.float64)


# --------------------------------------------------------------------------- linear
def linear_example_grad(A_i, G_i):
    """Per-example weight gradient of a linear layer, Eq. 4 summed over tokens.

    A_i: (T, d) inputs, G_i: (T, p) output gradients -> (p, d) = G_i^T A_i.
    """
    return _f64(G_i).T @ _f64(A_i)


def linear_sq_norms(A, G):
    """Squared Frobenius norm of every example's materialised gradient.

    A: (B, T, d), G: (B, T, p) -> (B,) float64.  Eq. 5 is the T = 1 case.
    """
    B = A.shape[0]
    out = np.zeros(B, dtype=np.float64)
    for i in range(B):
        P = linear_example_grad(A[i], G[i])
        out[i] = np.sum(P * P)
    return out


# ------------------------------------------------------------------------ embedding
def embed_example_grad(ids_i, G_i, V):
    """Per-example gradient of an embedding table: row ids_i[t] receives G_i[t].

    An embedding is a linear layer whose input is the one-hot row of the token,
    so Eq. 4 gives e_{id_t} g_t^T per token; repeated tokens add up.
    ids_i: (T,) ints in [0, V); G_i: (T, d) -> (V, d).
    """
    G_i = _f64(G_i)
    E = np.zeros((V, G_i.shape[1]), dtype=np.float64)
    for t in range(len(ids_i)):
        E[int(ids_i[t])] += G_i[t]
    return E


def embed_sq_norms(ids, G, V):
    """(B,) squared norms of the materialised per-example embedding gradients."""
    B = ids.shape[0]
    out = np.zeros(B, dtype=np.float64)
    for i in range(B):
        E = embed_example_grad(ids[i], G[i], V)
        out[i] = np.sum(E * E)
    return out


# ------------------------------------------------- vector parameters (bias, LayerNorm)
def vector_example_grad(G_i, X_i=None):
    """Per-example gradient of a parameter that acts element-wise along the feature axis.

    A bias b in z = W a + b receives delta_t per token (Eq. 4 with a constant input 1), so the
    example's gradient is sum_t G_i[t, :].  A LayerNorm gain gamma in y = gamma * xhat + beta
    receives sum_t G_i[t, :] * xhat_i[t, :] (G = gradient w.r.t. y); its beta is a bias.
    G_i: (T, p); X_i: (T, p) multiplier or None -> (p,).
    """
    G_i = _f64(G_i)
    out = np.zeros(G_i.shape[1], dtype=np.float64)
    for t in range(G_i.shape[0]):
        out += G_i[t] if X_i is None else G_i[t] * _f64(X_i[t])
    return out


def vector_sq_norms(G, X=None):
    """(B,) squared norms of the materialised per-example vector gradients."""
    B = G.shape[0]
    out = np.zeros(B, dtype=np.float64)
    for i in range(B):
        v = vector_example_grad(G[i], None if X is None else X[i])
        out[i] = np.sum(v * v)
    return out


def clipped_sum_vector(G, X, R):
    """sum_i R_i g_i for a vector parameter, (p,)."""
    acc = np.zeros(G.shape[2], dtype=np.float64)
    for i in range(G.shape[0]):
        acc += float(R[i]) * vector_example_grad(G[i], None if X is None else X[i])
    return acc


# ----------------------------------------------------------------------------- tied
def tied_sq_norms(ids, G_emb, A_lm, G_lm, V):
    """Shared embedding / LM-head matrix (Eq. 8): per-example norm of g_in + g_out.

    Returns a dict of (B,) arrays: 'in' = ||g_in||^2, 'out' = ||g_out||^2,
    'cross' = <g_in, g_out>, 'tied' = ||g_in + g_out||^2 taken on the
    materialised sum (left side of Eq. 11 / Eq. 13, not the right side).
    g_in: (V, d) embedding gradient; g_out = G_lm_i^T A_lm_i, also (V, d).
    """
    B = ids.shape[0]
    r = {k: np.zeros(B, dtype=np.float64) for k in ("in", "out", "cross", "tied")}
    for i in range(B):
        g_in = embed_example_grad(ids[i], G_emb[i], V)
        g_out = linear_example_grad(A_lm[i], G_lm[i])
        s = g_in + g_out
        r["in"][i] = np.sum(g_in * g_in)
        r["out"][i] = np.sum(g_out * g_out)
        r["cross"][i] = np.sum(g_in * g_out)
        r["tied"][i] = np.sum(s * s)
    return r


# ------------------------------------------------------------------------- clipping
def clip_factors(sq, C):
    """Eq. 2 / Eq. 7: norm_i = sqrt(sq_i), R_i = min(1, C / norm_i).

    No stabiliser is added (the paper has none); a zero norm gives R_i = 1.
    Returns (norms, R), both (B,) float64.
    """
    sq = _f64(sq)
    norms = np.sqrt(sq)
    R = np.ones_like(norms)
    for i in range(len(norms)):
        if norms[i] > 0.0:
            R[i] = min(1.0, float(C) / norms[i])
    return norms, R


def clipped_sum_linear(A, G, R):
    """sum_i R_i g_i over materialised per-example gradients (inner sum of Eq. 3)."""
    B = A.shape[0]
    acc = np.zeros((G.shape[2], A.shape[2]), dtype=np.float64)
    for i in range(B):
        acc += float(R[i]) * linear_example_grad(A[i], G[i])
    return acc


def clipped_sum_embed(ids, G, R, V):
    """sum_i R_i g_i for an embedding table, (V, d)."""
    B = ids.shape[0]
    acc = np.zeros((V, G.shape[2]), dtype=np.float64)
    for i in range(B):
        acc += float(R[i]) * embed_example_grad(ids[i], G[i], V)
    return acc


# ------------------------------------------------------------- integer side outputs
def first_occurrence(ids):
    """first[i, t] = smallest s with ids[i, s] == ids[i, t] (int32, brute force)."""
    ids = np.asarray(ids)
    B, T = ids.shape
    out = np.zeros((B, T), dtype=np.int32)
    for i in range(B):
        for t in range(T):
            s = 0
            while ids[i, s] != ids[i, t]:
                s += 1
            out[i, t] = s
    return out


def stable_token_sort(ids, V):
    """Stable counting sort of the flattened (B*T) ids.

    Returns perm (B*T,) int32, the flat positions ordered by token id and, among
    equal ids, by flat position; and seg (V+1,) int32 with seg[v] = number of
    positions whose id is < v.
    """
    flat = np.asarray(ids).reshape(-1)
    buckets = [[] for _ in range(V)]
    for pos in range(len(flat)):
        buckets[int(flat[pos])].append(pos)
    perm = np.zeros(len(flat), dtype=np.int32)
    seg = np.zeros(V + 1, dtype=np.int32)
    n = 0
    for v in range(V):
        seg[v] = n
        for pos in buckets[v]:
            perm[n] = pos
            n += 1
    seg[V] = n
    return perm, seg


# ------------------------------------------------------------------------ whole step
def dp_step(linears, ids, G_emb, V, C, lm=None, tied=False, positions=False,
            want_sums=True, vectors=()):
    """One DP-SGD clipping step over the parameter blocks it is handed.

    linears: list of (A, G) with A (B,T,d), G (B,T,p): the block linear layers.
    ids (B,T), G_emb (B,T,d): token embedding and the gradient reaching it.
    lm: (A_lm, G_lm) of the LM head or None.  tied: the head shares the
    embedding matrix (Eq. 8); then the embedding and head contributions enter
    through ||g_in + g_out||^2 (Eq. 13) and their clipped sums share one matrix.
    positions: also treat a learned position table (row t receives G_emb[i, t]).
    vectors: list of (G, X or None): biases and LayerNorm gains / shifts (see
    vector_example_grad); their clipped sums are returned as 'vector<k>'.

    Squared norms add over disjoint parameter blocks (Eq. 6, Eq. 10).
    Returns dict with 'sq', 'norms', 'clip', and (if want_sums) 'sums': a dict
    keyed 'linear<k>', 'wte', 'wpe', 'lm_head' (untied) or 'wte' holding the
    shared matrix (tied).
    """
    B, T = ids.shape
    sq = np.zeros(B, dtype=np.float64)
    for (A, G) in linears:
        sq += linear_sq_norms(A, G)
    for (G, X) in vectors:
        sq += vector_sq_norms(G, X)
    pos_ids = np.broadcast_to(np.arange(T), (B, T))
    if positions:
        sq += embed_sq_norms(pos_ids, G_emb, T)
    extra = {}
    if tied:
        assert lm is not None
        r = tied_sq_norms(ids, G_emb, lm[0], lm[1], V)
        sq += r["tied"]
        extra = {"sq_in": r["in"], "sq_out": r["out"], "cross": r["cross"]}
    else:
        sq += embed_sq_norms(ids, G_emb, V)
        if lm is not None:
            sq += linear_sq_norms(lm[0], lm[1])
    norms, R = clip_factors(sq, C)
    res = {"sq": sq, "norms": norms, "clip": R, **extra}
    if want_sums:
        sums = {}
        for k, (A, G) in enumerate(linears):
            sums[f"linear{k}"] = clipped_sum_linear(A, G, R)
        for k, (G, X) in enumerate(vectors):
            sums[f"vector{k}"] = clipped_sum_vector(G, X, R)
        if positions:
            sums["wpe"] = clipped_sum_embed(pos_ids, G_emb, R, T)
        wte = clipped_sum_embed(ids, G_emb, R, V)
        if lm is not None:
            head = clipped_sum_linear(lm[0], lm[1], R)
            if tied:
                wte = wte + head
            else:
                sums["lm_head"] = head
        sums["wte"] = wte
        res["sums"] = sums
    return res
