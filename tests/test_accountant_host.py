"""Host-side privacy accountant of the library against the quadrature oracle (no GPU needed: the
calls do no device work)."""
import pytest

from oracle import rdp_oracle as R
from paper_2609_40335_b200 import binding as dp


@pytest.mark.parametrize("q,sigma,steps,delta", [
    (24 / 67349, 0.62, 28062, 67349 ** -1.1),        # the shape of the paper's SST-2 runs (B = 24)
    (24 / 67349, 1.0, 11225, 67349 ** -1.1),
    (0.01, 1.1, 1000, 1e-5),
    (0.25, 2.0, 40, 1e-6),
    (1.0, 4.0, 3, 1e-5),
    (0.0, 0.7, 100, 1e-5),
])
def test_epsilon_matches_the_quadrature_oracle(q, sigma, steps, delta):
    got, order = dp.dp_rdp_epsilon(q, sigma, steps, delta)
    want, want_order = R.epsilon(q, sigma, steps, delta)
    assert got == pytest.approx(want, rel=1e-7, abs=1e-8)
    assert abs(order - want_order) <= 1                 # near-ties between neighbouring orders


def test_sigma_search_meets_the_paper_budget():
    q, steps, delta = 24 / 67349, 28062, 67349 ** -1.1
    for target in (1.0, 3.0, 5.0):                       # the three budgets the paper evaluates
        s = dp.dp_sigma_for_epsilon(q, steps, target, delta, 1e-5)
        assert R.epsilon(q, s, steps, delta)[0] <= target + 1e-6
        assert R.epsilon(q, s - 5e-5, steps, delta)[0] > target - 1e-4
    s1, s3, s5 = (dp.dp_sigma_for_epsilon(q, steps, t, delta) for t in (1.0, 3.0, 5.0))
    assert s1 > s3 > s5 > 0.3                            # tighter budget, more noise


def test_sigma_search_agrees_with_the_oracle_search():
    q, steps, delta = 0.02, 500, 1e-5
    assert dp.dp_sigma_for_epsilon(q, steps, 2.0, delta, 1e-5) == pytest.approx(
        R.sigma_for_epsilon(q, steps, 2.0, delta, tol=1e-5), abs=3e-5)


def test_accountant_rejects_bad_arguments():
    for bad in [(-0.1, 1.0, 10, 1e-5), (1.5, 1.0, 10, 1e-5), (0.1, 0.0, 10, 1e-5), (0.1, 1.0, -1, 1e-5),
                (0.1, 1.0, 10, 0.0), (0.1, 1.0, 10, 1.0)]:
        with pytest.raises(dp.DpGhostError):
            dp.dp_rdp_epsilon(*bad)
    with pytest.raises(dp.DpGhostError):                 # below the floor of the conversion term
        dp.dp_sigma_for_epsilon(0.01, 100, 1e-3, 1e-5)
