// Host-side privacy accounting: the noise multiplier sigma of Eq. 3 from a target (epsilon, delta),
// the sampling rate and the number of steps, as the paper's setup does with a Renyi-DP accountant
// (target epsilon = 3, delta = N^-1.1).  No device code: plain C++ compiled into the same library.
//
// One DP-SGD step is the Poisson-subsampled Gaussian mechanism with sensitivity 1 (per-example
// gradients are clipped to C and the noise has standard deviation sigma*C).  For an INTEGER order
// alpha its Renyi divergence has the finite binomial form
//     A(alpha) = sum_{k=0..alpha} C(alpha,k) (1-q)^(alpha-k) q^k exp((k^2 - k) / (2 sigma^2)),
//     eps_RDP(alpha) = log A(alpha) / (alpha - 1),
// RDP adds over steps, and epsilon(delta) = min_alpha steps*eps_RDP(alpha) + log(1/delta)/(alpha-1).
// The sum is evaluated in log space (the last terms overflow otherwise).  Orders 2 .. 256.
#include <cmath>
#include <limits>
#include <vector>

#include "../../include/dp_ghost.h"

namespace {

constexpr int kMinOrder = 2, kMaxOrder = 256;

double log_add(double a, double b) {
  if (a == -std::numeric_limits<double>::infinity()) return b;
  if (b == -std::numeric_limits<double>::infinity()) return a;
  const double m = a > b ? a : b;
  return m + std::log1p(std::exp(-std::fabs(a - b)));
}

// log A(alpha) for integer alpha >= 2
double log_moment(double q, double sigma, int alpha) {
  if (q == 0.0) return 0.0;
  if (q == 1.0) return double(alpha) * (alpha - 1) / (2.0 * sigma * sigma);
  const double lq = std::log(q), l1q = std::log1p(-q);
  double acc = -std::numeric_limits<double>::infinity();
  for (int k = 0; k <= alpha; ++k) {
    const double log_binom = std::lgamma(alpha + 1.0) - std::lgamma(k + 1.0) - std::lgamma(alpha - k + 1.0);
    const double term = log_binom + k * lq + (alpha - k) * l1q + double(k) * (k - 1) / (2.0 * sigma * sigma);
    acc = log_add(acc, term);
  }
  return acc;
}

bool args_ok(double q, double sigma, long long steps, double delta) {
  return q >= 0.0 && q <= 1.0 && sigma > 0.0 && std::isfinite(sigma) && steps >= 0 && delta > 0.0 &&
         delta < 1.0;
}

double epsilon_of(double q, double sigma, long long steps, double delta, int* best_order) {
  double best = std::numeric_limits<double>::infinity();
  int arg = kMinOrder;
  for (int a = kMinOrder; a <= kMaxOrder; ++a) {
    const double e = double(steps) * log_moment(q, sigma, a) / (a - 1.0) + std::log(1.0 / delta) / (a - 1.0);
    if (e < best) { best = e; arg = a; }
  }
  if (best_order) *best_order = arg;
  return best;
}

}  // namespace

extern "C" {

dp_status dp_rdp_epsilon(double q, double sigma, int64_t steps, double delta, double* epsilon,
                         int32_t* best_order) {
  if (!epsilon || !args_ok(q, sigma, steps, delta)) return DP_ERR_INVALID_ARG;
  int order = 0;
  *epsilon = epsilon_of(q, sigma, steps, delta, &order);
  if (best_order) *best_order = order;
  return DP_OK;
}

dp_status dp_sigma_for_epsilon(double q, int64_t steps, double target_epsilon, double delta,
                               double tolerance, double* sigma) {
  if (!sigma || !(target_epsilon > 0.0) || !(tolerance > 0.0) || !args_ok(q, 1.0, steps, delta))
    return DP_ERR_INVALID_ARG;
  // even without any step, the conversion leaves log(1/delta)/(alpha_max - 1): below it no sigma works
  if (target_epsilon <= std::log(1.0 / delta) / (kMaxOrder - 1.0)) return DP_ERR_UNSUPPORTED;
  double lo = 0.3, hi = 1.0;
  int guard = 0;
  while (epsilon_of(q, hi, steps, delta, nullptr) > target_epsilon) {
    hi *= 2.0;
    if (++guard > 60) return DP_ERR_UNSUPPORTED;
  }
  while (lo > 1e-3 && epsilon_of(q, lo, steps, delta, nullptr) < target_epsilon) lo *= 0.5;
  while (hi - lo > tolerance) {                 // epsilon decreases as sigma grows
    const double mid = 0.5 * (lo + hi);
    if (epsilon_of(q, mid, steps, delta, nullptr) > target_epsilon) lo = mid;
    else hi = mid;
  }
  *sigma = hi;
  return DP_OK;
}

}  // extern "C"
