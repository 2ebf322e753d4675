"""Float64 CPU oracle of the Gaussian noise of Eq. 3, N(0, sigma^2 C^2 I).

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA path.

The paper fixes only the distribution.  To make the draw reproducible and
independent of how a device splits the work, the noise is defined as a pure
function of (seed, tensor_id, step, element index j):

  * generator: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11);
    key = (seed & 0xffffffff, seed >> 32); counter = (q & 0xffffffff, q >> 32,
    tensor_id, step) with q = j // 4; the four output words x0..x3 serve
    elements 4q .. 4q+3.
  * Box-Muller on the word pairs (x0, x1) and (x2, x3):
      u1 = ((xa >> 8) + 1) * 2^-24  in (0, 1],   u2 = (xb >> 8) * 2^-24 in [0, 1)
      r  = sqrt(-2 ln u1),  z_a = r cos(2 pi u2),  z_b = r sin(2 pi u2)
    so element 4q+0 = z_a(x0,x1), 4q+1 = z_b(x0,x1), 4q+2 = z_a(x2,x3),
    4q+3 = z_b(x2,x3).
  * result[j] = scale * (x[j] + sigma * C * z[j])   (scale = 1/|B| gives Eq. 3).

Pins (tests/test_oracle_noise.py): the published Philox4x32-10 known-answer
vectors (tests/golden/philox4x32_10_kat.txt), agreement of the vectorised
generator with a scalar pure-integer one, moments / Kolmogorov-Smirnov against
the normal law, and stream-separation properties.
"""
from __future__ import annotations

import math

import numpy as np

_M0 = 0xD2511F53
_M1 = 0xCD9E8D57
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10_scalar(counter, key):
    """One Philox4x32-10 block with Python integers. counter: 4 words, key: 2 words."""
    c0, c1, c2, c3 = (int(c) & _MASK for c in counter)
    k0, k1 = (int(k) & _MASK for k in key)
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK
        hi1, lo1 = p1 >> 32, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0), lo1, (hi0 ^ c3 ^ k1), lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Vectorised Philox4x32-10: uint64 arrays holding 32-bit words -> four uint64 arrays."""
    c0 = np.asarray(c0, dtype=np.uint64).copy()
    c1 = np.asarray(c1, dtype=np.uint64).copy()
    c2 = np.asarray(c2, dtype=np.uint64).copy()
    c3 = np.asarray(c3, dtype=np.uint64).copy()
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = int(k0) & _MASK
    k1 = int(k1) & _MASK
    m = np.uint64(_MASK)
    s32 = np.uint64(32)
    for _ in range(10):
        p0 = np.uint64(_M0) * c0
        p1 = np.uint64(_M1) * c2
        hi0, lo0 = p0 >> s32, p0 & m
        hi1, lo1 = p1 >> s32, p1 & m
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def _box_muller(xa, xb):
    u1 = ((xa >> np.uint64(8)).astype(np.float64) + 1.0) * (2.0 ** -24)
    u2 = (xb >> np.uint64(8)).astype(np.float64) * (2.0 ** -24)
    r = np.sqrt(-2.0 * np.log(u1))
    ang = 2.0 * math.pi * u2
    return r * np.cos(ang), r * np.sin(ang)


def standard_normals(n, seed, tensor_id, step, start=0):
    """z[start : start+n] of the stream (seed, tensor_id, step), float64."""
    n = int(n)
    start = int(start)
    if n == 0:
        return np.zeros(0, dtype=np.float64)
    q_lo = start // 4
    q_hi = (start + n - 1) // 4
    q = np.arange(q_lo, q_hi + 1, dtype=np.uint64)
    x0, x1, x2, x3 = philox4x32_10(q & np.uint64(_MASK), q >> np.uint64(32),
                                   np.uint64(int(tensor_id) & _MASK),
                                   np.uint64(int(step) & _MASK),
                                   int(seed) & _MASK, (int(seed) >> 32) & _MASK)
    za, zb = _box_muller(x0, x1)
    zc, zd = _box_muller(x2, x3)
    z = np.stack([za, zb, zc, zd], axis=1).reshape(-1)
    off = start - 4 * q_lo
    return z[off:off + n]


def add_noise(x, sigma, C, scale, seed, tensor_id, step):
    """Eq. 3 on one parameter tensor: scale * (x + sigma*C*z), flat row-major order."""
    x = np.asarray(x, dtype=np.float64)
    z = standard_normals(x.size, seed, tensor_id, step).reshape(x.shape)
    return float(scale) * (x + float(sigma) * float(C) * z)
