"""Pins for oracle/noise_oracle.py: published Philox known answers, scalar-vs-vector
agreement, the normal law (moments, Kolmogorov-Smirnov), stream separation."""
import math
import os

import numpy as np
from scipy import stats

from oracle import noise_oracle as N


def _kat_rows():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            w = [int(x, 16) for x in line.split()]
            yield w[:4], w[4:6], w[6:]


def test_philox_known_answers_scalar_and_vector():
    n = 0
    for ctr, key, out in _kat_rows():
        assert list(N.philox4x32_10_scalar(ctr, key)) == out
        v = N.philox4x32_10(*[np.array([c], dtype=np.uint64) for c in ctr], key[0], key[1])
        assert [int(x[0]) for x in v] == out
        n += 1
    assert n == 3


def test_vector_matches_scalar_on_random_counters():
    rng = np.random.default_rng(5)
    ctr = rng.integers(0, 2 ** 32, size=(64, 4), dtype=np.uint64)
    k0, k1 = 0x12345678, 0x9ABCDEF0
    v = N.philox4x32_10(ctr[:, 0], ctr[:, 1], ctr[:, 2], ctr[:, 3], k0, k1)
    for r in range(64):
        assert tuple(int(x[r]) for x in v) == N.philox4x32_10_scalar(ctr[r], (k0, k1))


def test_element_layout_and_box_muller_by_hand():
    seed, tid, step = (0xDEADBEEF << 32) | 0x1234, 3, 9
    z = N.standard_normals(10, seed, tid, step)
    for q in range(2):
        x = N.philox4x32_10_scalar((q, 0, tid, step), (0x1234, 0xDEADBEEF))
        for pair in range(2):
            xa, xb = x[2 * pair], x[2 * pair + 1]
            u1 = ((xa >> 8) + 1) / 2 ** 24
            u2 = (xb >> 8) / 2 ** 24
            r = math.sqrt(-2 * math.log(u1))
            assert abs(z[4 * q + 2 * pair] - r * math.cos(2 * math.pi * u2)) < 1e-14
            assert abs(z[4 * q + 2 * pair + 1] - r * math.sin(2 * math.pi * u2)) < 1e-14
    # a window of the stream equals the same window of a longer draw
    np.testing.assert_array_equal(N.standard_normals(5, seed, tid, step, start=3), z[3:8])


def test_normal_law():
    z = N.standard_normals(4_000_000, seed=42, tensor_id=0, step=0)
    assert abs(z.mean()) < 4 / math.sqrt(z.size)
    assert abs(z.var() - 1) < 4 * math.sqrt(2 / z.size)
    assert abs(stats.kurtosis(z)) < 0.02 and abs(stats.skew(z)) < 0.01
    assert np.abs(z).max() < math.sqrt(2 * 24 * math.log(2)) + 1e-9       # u1 >= 2^-24
    assert stats.kstest(z[:500_000], "norm").pvalue > 1e-3
    # neighbours are uncorrelated, also across the (cos, sin) pairs
    for lag in (1, 2, 3, 4):
        assert abs(np.corrcoef(z[:-lag], z[lag:])[0, 1]) < 5 / math.sqrt(z.size)


def test_streams_and_noise_application():
    a = N.standard_normals(1000, 1, 0, 0)
    assert not np.array_equal(a, N.standard_normals(1000, 1, 1, 0))
    assert not np.array_equal(a, N.standard_normals(1000, 1, 0, 1))
    assert not np.array_equal(a, N.standard_normals(1000, 2, 0, 0))
    assert not np.array_equal(a, N.standard_normals(1000, 1 << 32, 0, 0))
    np.testing.assert_array_equal(a, N.standard_normals(1000, 1, 0, 0))
    x = np.arange(12, dtype=np.float64).reshape(3, 4)
    np.testing.assert_array_equal(N.add_noise(x, 0.0, 1.0, 1.0, 1, 0, 0), x)
    y = N.add_noise(x, 0.8, 0.5, 0.25, 1, 0, 0)
    np.testing.assert_allclose(y, 0.25 * (x + 0.4 * a[:12].reshape(3, 4)), rtol=1e-15)
