// Host side of Algorithm 1 (steps 2, 5-9) and Algorithm 2 (steps 2-6), and the cumulative
// table of the noise law (Def. 3.3, Eq. 2).  IEEE doubles, fixed evaluation order, compiled
// without contraction or fast-math so that the result is reproducible bit for bit.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "isc_internal.h"

namespace isc {

namespace {

// log of the binomial coefficient C(n, i)
inline double log_choose(int64_t n, int64_t i)
{
    return std::lgamma((double)n + 1.0) - std::lgamma((double)i + 1.0) - std::lgamma((double)(n - i) + 1.0);
}

// P[Binomial(n, p) >= k], terms added for i = k, k+1, ..., n; log_c[i - k] = log_choose(n, i), computed once per
// bound (the same value in the same place of the same expression, so the sum is what it was term by term)
double upper_tail(int64_t k, int64_t n, double p, const std::vector<double> &log_c)
{
    const double log_p = std::log(p);
    const double log_q = std::log1p(-p);
    double total = 0.0;
    for (int64_t i = k; i <= n; ++i)
        total += std::exp(log_c[(size_t)(i - k)] + (double)i * log_p + (double)(n - i) * log_q);
    return total;
}

inline int first_max(const int32_t *v, int n)
{
    int arg = 0;
    for (int i = 1; i < n; ++i)
        if (v[i] > v[arg]) arg = i;
    return arg;
}

}  // namespace

// One-sided (1 - alpha) Clopper-Pearson lower bound (Algorithm 1, step 5): the success
// probability at which seeing k or more successes in n trials has probability alpha.
double lower_conf_bound(int64_t k, int64_t n, double alpha)
{
    if (k <= 0) return 0.0;
    if (k >= n) return std::exp(std::log(alpha) / (double)n);
    std::vector<double> log_c((size_t)(n - k + 1));
    for (int64_t i = k; i <= n; ++i) log_c[(size_t)(i - k)] = log_choose(n, i);
    double left = 0.0, right = (double)k / (double)n;
    for (int step = 0; step < 64; ++step) {
        const double mid = 0.5 * (left + right);
        if (upper_tail(k, n, mid, log_c) < alpha)
            left = mid;
        else
            right = mid;
    }
    return left;
}

// Phi^-1(p) for p >= 1/2 (Algorithm 1, step 7) by bisection of Phi(x) = erfc(-x/sqrt 2)/2 on [0, 9].
double normal_quantile(double p)
{
    double left = 0.0, right = 9.0;
    for (int step = 0; step < 64; ++step) {
        const double mid = 0.5 * (left + right);
        const double cdf = 0.5 * std::erfc(-mid / std::sqrt(2.0));
        if (cdf < p)
            left = mid;
        else
            right = mid;
    }
    return left;
}

// Two-sided exact binomial test of n_a successes out of m at probability 1/2 (Algorithm 2, step 3).
double binom_pvalue_half(int64_t n_a, int64_t m)
{
    double total = 0.0;
    for (int64_t i = n_a; i <= m; ++i)
        total += std::exp(log_choose(m, i) - (double)m * std::log(2.0));
    const double pv = 2.0 * total;
    return pv < 1.0 ? pv : 1.0;
}

int32_t decide_certify(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N,
                       double sigma, double alpha, double *radius, double *p_lower)
{
    const int c_a = first_max(counts0, n_classes);          // step 2: label with the most selection votes
    const int64_t n_a = counts[c_a];                        // step 4: its votes among the N fresh samples
    const double p_a = lower_conf_bound(n_a, N, alpha);     // step 5
    if (p_lower) *p_lower = p_a;
    if (p_a > 0.5) {                                        // steps 6-7
        *radius = sigma * normal_quantile(p_a);
        return c_a;
    }
    *radius = 0.0;                                          // step 8: ABSTAIN
    return -1;
}

namespace {

// floor(p * 2^32) as the table's fixed-point probability, saturated to 32 bits
uint32_t to_fixed32(double p)
{
    const double scaled = std::floor(p * 4294967296.0);
    if (scaled <= 0.0) return 0u;
    return scaled >= 4294967295.0 ? 4294967295u : (uint32_t)scaled;
}

// Theorem 3.2 step 2: the quantile of the discrete Gaussian by lookup, the first level whose cumulative entry reaches p
int32_t table_quantile(const std::vector<uint32_t> &cum, uint32_t p_fx)
{
    const int32_t T = (int32_t)(cum.size() - 1) / 2;
    const int32_t at = (int32_t)(std::lower_bound(cum.begin(), cum.end(), p_fx) - cum.begin());
    return at > 2 * T ? T : at - T;
}

}  // namespace

int32_t decide_certify_integer(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N, double sigma,
                               double alpha, bool two_sided, int32_t *q, int64_t *q_squared)
{
    *q = 0; *q_squared = 0;
    const int c_a = first_max(counts0, n_classes);           // Algorithm 1 steps 2, 4, 5, 6
    const double p_a = lower_conf_bound(counts[c_a], N, alpha);
    if (!(p_a > 0.5)) return -1;
    std::vector<uint32_t> cum;
    noise_table(sigma, cum);
    const int32_t q_a = table_quantile(cum, to_fixed32(p_a));
    if (!two_sided) {                                         // Theorem 3.2 steps 2-3: radius and squared radius in pixel levels
        *q = q_a;
        *q_squared = (int64_t)q_a * q_a;
        return c_a;
    }
    // Theorem 3.1: the runner-up's upper bound enters as well; d = q_A - q_B is twice the radius
    int64_t n_b = 0;
    for (int c = 0; c < n_classes; ++c)
        if (c != c_a && counts[c] > n_b) n_b = counts[c];
    const double p_b = 1.0 - lower_conf_bound(N - n_b, N, alpha);
    if (p_a < p_b) return -1;
    const int32_t d = q_a - table_quantile(cum, to_fixed32(p_b));
    *q = d;
    *q_squared = (int64_t)d * d;
    return c_a;
}

int32_t decide_predict(const int32_t *counts, int n_classes, double alpha)
{
    const int c_a = first_max(counts, n_classes);
    const int64_t n_a = counts[c_a];
    int64_t n_b = 0;
    bool seen = false;
    for (int c = 0; c < n_classes; ++c) {
        if (c == c_a) continue;
        if (!seen || counts[c] > n_b) { n_b = counts[c]; seen = true; }
    }
    return binom_pvalue_half(n_a, n_a + n_b) <= alpha ? c_a : -1;
}

int noise_halfwidth(double sigma)
{
    return (int)std::ceil(7.0 * (255.0 * sigma));
}

// cum[z + T] = floor(2^32 * P[Z <= z]) for the discrete Gaussian of Eq. 2 on the integer pixel
// levels with std 255*sigma, support cut at +-T; the last entry is 2^32 - 1.
void noise_table(double sigma, std::vector<uint32_t> &cum)
{
    const double s = 255.0 * sigma;
    const int T = noise_halfwidth(sigma);
    const double two_var = 2.0 * s * s;
    std::vector<double> weight((size_t)(2 * T + 1));
    double norm = 0.0;
    for (int z = -T; z <= T; ++z) {
        weight[(size_t)(z + T)] = std::exp(-(double)((int64_t)z * z) / two_var);
        norm += weight[(size_t)(z + T)];
    }
    cum.resize((size_t)(2 * T + 1));
    double running = 0.0;
    for (int z = -T; z <= T; ++z) {
        running += weight[(size_t)(z + T)];
        double scaled = std::floor(running / norm * 4294967296.0);
        if (scaled > 4294967295.0) scaled = 4294967295.0;
        cum[(size_t)(z + T)] = (uint32_t)scaled;
    }
    cum[(size_t)(2 * T)] = 4294967295u;
}

// The same table form for the rounded continuous Gaussian: delta = round(255 sigma g), g ~ N(0, 1), the noise of the
// paper's comparison method that perturbs with continuous noise and then quantises (Sec. 4.1, comparison methods):
// cum[z + T] = floor(2^32 * Phi((z + 1/2) / (255 sigma))).
void noise_table_rounded(double sigma, std::vector<uint32_t> &cum)
{
    const double s = 255.0 * sigma;
    const int T = noise_halfwidth(sigma);
    cum.resize((size_t)(2 * T + 1));
    for (int z = -T; z <= T; ++z) {
        const double cdf = 0.5 * std::erfc(-(((double)z + 0.5) / s) / std::sqrt(2.0));
        double scaled = std::floor(cdf * 4294967296.0);
        if (scaled > 4294967295.0) scaled = 4294967295.0;
        cum[(size_t)(z + T)] = (uint32_t)scaled;
    }
    cum[(size_t)(2 * T)] = 4294967295u;
}

}  // namespace isc
