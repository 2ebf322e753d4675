"""Privacy accounting oracle (test infrastructure only: the product never imports this).

The paper calibrates the noise multiplier sigma from a target (epsilon, delta) with a Renyi-DP
accountant (Section "Experimental setup": target epsilon = 3, delta = N^-1.1, sampling rate and
number of steps given).  This file writes the DEFINITIONS out, in float64, by numerical quadrature:

  * the Renyi divergence of order alpha between the Poisson-subsampled Gaussian mechanism
    (1-q) N(0, sigma^2) + q N(1, sigma^2) and N(0, sigma^2)  (sensitivity 1 after clipping, Eq. 2-3),
        A(alpha) = E_{x ~ N(0, sigma^2)} [ ((1-q) + q exp((2x-1) / (2 sigma^2)))^alpha ],
        eps_RDP(alpha) = log A(alpha) / (alpha - 1);
  * composition over `steps` identical steps: RDP adds;
  * conversion to (epsilon, delta): epsilon = min over orders of
        steps * eps_RDP(alpha) + log(1/delta) / (alpha - 1).

Reading taken where the paper is silent (it only names the accountant): integer orders
alpha = 2 .. 256, the conversion above (the classical one).  Pinned by closed forms in
tests/test_oracle_rdp.py: q = 1 gives alpha / (2 sigma^2); alpha = 2 gives
log(1 + q^2 (exp(1/sigma^2) - 1)); q = 0 gives 0; monotonicity in q, sigma and steps.
"""
import numpy as np

ORDERS = tuple(range(2, 257))


def log_moment(q, sigma, alpha, points_per_sigma=400):
    """log A(alpha) by the trapezoid rule on a grid wide enough for both mixture components."""
    q, sigma, alpha = float(q), float(sigma), float(alpha)
    if q == 0.0:
        return 0.0
    # the integrand is a mixture of Gaussians with means 0 .. alpha: cover them with 12 sigma to spare
    lo, hi = -12.0 * sigma, alpha + 12.0 * sigma
    n = int((hi - lo) / sigma * points_per_sigma) + 1
    x = np.linspace(lo, hi, n)
    log_base = -x * x / (2 * sigma * sigma) - np.log(sigma * np.sqrt(2 * np.pi))
    log_ratio_term = (2 * x - 1) / (2 * sigma * sigma)
    if q == 1.0:
        log_mix = log_ratio_term
    else:
        log_mix = np.logaddexp(np.log1p(-q), np.log(q) + log_ratio_term)
    f = log_base + alpha * log_mix
    m = f.max()
    w = np.exp(f - m)
    integral = (w.sum() - 0.5 * (w[0] + w[-1])) * (x[1] - x[0])
    return float(m + np.log(integral))


def rdp(q, sigma, alpha):
    """eps_RDP(alpha) of one step."""
    return log_moment(q, sigma, alpha) / (alpha - 1.0)


def epsilon(q, sigma, steps, delta, orders=ORDERS):
    """(epsilon, best order) after `steps` steps."""
    best, best_a = np.inf, None
    for a in orders:
        e = steps * rdp(q, sigma, a) + np.log(1.0 / delta) / (a - 1.0)
        if e < best:
            best, best_a = e, a
    return float(best), best_a


def sigma_for_epsilon(q, steps, target_eps, delta, orders=ORDERS, tol=1e-6):
    """Smallest sigma (to `tol`) whose epsilon does not exceed the target: bisection, epsilon is
    decreasing in sigma."""
    lo, hi = 0.3, 1.0
    while epsilon(q, hi, steps, delta, orders)[0] > target_eps:
        hi *= 2.0
    while epsilon(q, lo, steps, delta, orders)[0] < target_eps and lo > 1e-3:
        lo *= 0.5
    while hi - lo > tol:
        mid = 0.5 * (lo + hi)
        if epsilon(q, mid, steps, delta, orders)[0] > target_eps:
            lo = mid
        else:
            hi = mid
    return hi
