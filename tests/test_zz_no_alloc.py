"""dp_embed_norms_static: the embedding norm for callers that cannot allocate (its scratch is a
fixed array inside the library).  Checked through the C ABI against dp_embed_norms, and against
the float64 oracle's materialised embedding gradient, on two calls in a row; collected last so
that a run stopping at the first failure has run everything else."""
import numpy as np
import pytest
import torch

from oracle import dp_oracle as O
from paper_2609_40335_b200 import binding as dp
from paper_2609_40335_b200 import pipeline as P
from paper_2609_40335_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    dev = torch.device("cuda:0")
    L = dp.load()
    for call, (B, T, d, V, seed) in enumerate([(32, 128, 768, 50257, 1), (5, 300, 200, 977, 2)]):
        ids = torch.from_numpy(W.zipf_ids(B, T, V, 1.1, seed)).to(dev)
        G = P.to_device(W._normal((B, T, d), 1e-2, "bf16", seed + 10))
        ref = torch.zeros(B, device=dev)
        fo_ref = torch.full((B, T), -1, dtype=torch.int32, device=dev)
        dp.dp_embed_norms(ids, G, V, ref, first_occ=fo_ref)
        got = torch.full((B,), 0.5, device=dev)              # += semantics: starts non-zero
        fo = torch.full((B, T), -1, dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        before = torch.cuda.memory_allocated(dev)
        # straight through the C ABI: device pointers and sizes only, no workspace argument
        rc = L.dp_embed_norms_static(ids.data_ptr(), G.data_ptr(), G.stride(-2), dp.DP_BF16, B, T, d, V,
                                     got.data_ptr(), fo.data_ptr(), status.data_ptr(),
                                     torch.cuda.current_stream().cuda_stream)
        assert rc == 0, L.dp_status_string(rc)
        assert torch.cuda.memory_allocated(dev) == before    # nothing was allocated through torch
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        err = ((got - 0.5) - ref).abs() / ref
        assert float(err.max()) < 2e-3, (call, err)
        assert torch.equal(fo, fo_ref)
        # and the oracle: the (V, d) embedding gradient of every example, materialised in float64
        ids_h = ids.cpu().numpy()
        G_h = G.float().cpu().numpy().astype(np.float64)
        want = O.embed_sq_norms(ids_h, G_h, V)
        assert np.abs((got.cpu().numpy() - 0.5) - want).max() / want.max() < 2e-3, call
        assert np.array_equal(fo.cpu().numpy(), O.first_occurrence(ids_h))
    # sizes beyond the built-in array are refused with their own status, nothing is enqueued
    B, T, d = 1024, 8, 8192                                  # 1024 * 32 slabs > 16384 floats
    ids = torch.zeros(B, T, dtype=torch.int32, device=dev)
    G = torch.zeros(B, T, d, dtype=torch.bfloat16, device=dev)
    sq = torch.zeros(B, device=dev)
    with pytest.raises(dp.DpGhostError) as e:
        dp.dp_embed_norms_static(ids, G, 10, sq)
    assert e.value.status == 6 and "scratch" in str(e.value)
