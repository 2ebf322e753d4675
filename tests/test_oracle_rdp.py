"""Pins of the accounting oracle (closed forms and invariants; no GPU)."""
import math

import numpy as np
import pytest

from oracle import rdp_oracle as R


@pytest.mark.parametrize("sigma", [0.5, 0.8, 1.0, 2.5])
@pytest.mark.parametrize("alpha", [2, 3, 8, 32, 100])
def test_full_batch_is_the_gaussian_mechanism(sigma, alpha):
    # q = 1: Renyi divergence between N(1, s^2) and N(0, s^2) is alpha / (2 s^2)
    assert R.rdp(1.0, sigma, alpha) == pytest.approx(alpha / (2 * sigma * sigma), rel=1e-9)


@pytest.mark.parametrize("q", [1e-4, 3.6e-4, 0.01, 0.3])
@pytest.mark.parametrize("sigma", [0.6, 1.0, 1.7])
def test_order_two_closed_form(q, sigma):
    # E[((1-q) + q L)^2] with E[L] = 1, E[L^2] = exp(1/s^2)
    want = math.log1p(q * q * math.expm1(1.0 / (sigma * sigma)))
    # the quadrature is good to ~1e-13 absolute in log A, which is all a tiny q leaves to see
    assert R.rdp(q, sigma, 2) == pytest.approx(want, rel=1e-8, abs=5e-13)


@pytest.mark.parametrize("q,sigma", [(0.01, 0.7), (0.2, 1.1)])
def test_order_three_closed_form(q, sigma):
    # third moment of the likelihood ratio: E[L^3] = exp(3/s^2)
    e1, e3 = math.exp(1 / sigma ** 2), math.exp(3 / sigma ** 2)
    a3 = (1 - q) ** 3 + 3 * (1 - q) ** 2 * q + 3 * (1 - q) * q * q * e1 + q ** 3 * e3
    assert R.rdp(q, sigma, 3) == pytest.approx(math.log(a3) / 2, rel=1e-8)


def test_no_sampling_no_loss_and_monotonicity():
    assert R.rdp(0.0, 1.0, 8) == 0.0
    assert R.rdp(0.01, 1.0, 8) < R.rdp(0.02, 1.0, 8)            # more sampling, more loss
    assert R.rdp(0.01, 1.2, 8) < R.rdp(0.01, 1.0, 8)            # more noise, less loss
    assert R.rdp(0.01, 1.0, 4) < R.rdp(0.01, 1.0, 8)            # Renyi divergence grows with the order
    e1, _ = R.epsilon(0.01, 1.0, 100, 1e-5)
    e2, _ = R.epsilon(0.01, 1.0, 200, 1e-5)
    assert 0 < e1 < e2 < 2 * e1 + 1e-9                          # composition: at most additive


def test_gaussian_mechanism_epsilon_in_closed_form():
    # q = 1, one step: minimise alpha/(2 s^2) + log(1/delta)/(alpha-1) over integer orders
    s, delta = 2.0, 1e-6
    want = min(a / (2 * s * s) + math.log(1 / delta) / (a - 1) for a in R.ORDERS)
    got, order = R.epsilon(1.0, s, 1, delta)
    assert got == pytest.approx(want, rel=1e-9)
    a_star = 1 + math.sqrt(2 * s * s * math.log(1 / delta))     # continuous minimiser
    assert abs(order - a_star) <= 1.0


def test_sigma_search_inverts_epsilon():
    q, steps, delta = 24 / 67349, 28062, 67349 ** -1.1          # the shape of the paper's SST-2 runs
    s = R.sigma_for_epsilon(q, steps, 3.0, delta, tol=1e-4)
    assert R.epsilon(q, s, steps, delta)[0] <= 3.0 < R.epsilon(q, s - 2e-4, steps, delta)[0]
    assert 0.4 < s < 1.5
