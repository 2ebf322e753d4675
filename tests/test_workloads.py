"""Host-side checks of the seeded input generators (no method arithmetic there)."""
import numpy as np
import torch

from paper_2609_40335_b200 import workloads as W


def test_bf16_rounding_matches_library_rne():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32) * 1e-2,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38], dtype=np.float32)])
    bits = W.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, want)
    back = W.bf16_bits_to_f32(bits)
    np.testing.assert_array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_zipf_is_bounded_and_head_heavy():
    ids = W.zipf_ids(64, 512, W.GPT2_VOCAB, 1.1, seed=1)
    assert ids.min() >= 0 and ids.max() < W.GPT2_VOCAB and ids.dtype == np.int32
    w = np.arange(1, W.GPT2_VOCAB + 1) ** -1.1
    p0 = w[0] / w.sum()
    frac0 = (ids == 0).mean()
    assert abs(frac0 - p0) < 5 * np.sqrt(p0 / ids.size)
    assert 0.12 < p0 < 0.16


def test_named_workloads_are_seeded_and_shaped():
    a = W.named_workload("cfg1")
    b = W.named_workload("cfg1")
    assert a.dtype == "f32" and a.B == 4 and a.T == 16 and a.V == 1000 and a.lm is None
    assert a.linears[0].A.data.shape == (4, 16, 64)
    np.testing.assert_array_equal(a.linears[0].G.data, b.linears[0].G.data)
    np.testing.assert_array_equal(a.ids, b.ids)
    assert not np.array_equal(a.ids, W.named_workload("cfg1", seed=1).ids)
    s = W.named_workload("cfg2", B=2, T=8, n_blocks=1, V=1003)
    assert [(l.d, l.p) for l in s.linears] == [(768, 2304), (768, 768), (768, 3072), (3072, 768)]
    assert s.lm.G.ld == 1008 and s.lm.G.cols == 1003 and s.lm.G.widened().shape == (2, 8, 1003)
    pad = W.bf16_bits_to_f32(s.lm.G.data[..., 1003:])
    assert np.isnan(pad).all()                      # padding must never be read
    g = s.linears[0].G.widened()
    assert 0.008 < g.std() < 0.012                  # N(0, 1e-4) read as variance
