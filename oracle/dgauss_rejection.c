/*
 * dgauss_rejection.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A second, table-free sampler of the discrete Gaussian N_Z(0, s^2) (Def. 3.3, Eq. 2), used only to pin the
 * table sampler of intrs_oracle.c against something that is not a table: the rejection sampler the paper points to
 * for its noise (Sec. 3.3: it follows the sampling strategy of Canonne, Kamath and Steinke, "The Discrete Gaussian
 * for Differential Privacy", 2020).  Restated from that publication:
 *
 *   t = floor(s) + 1
 *   repeat
 *     discrete Laplace Y with scale t:
 *       repeat  U uniform on {0..t-1};  keep it with probability exp(-U/t)  until kept
 *       V = number of successes before the first failure of Bernoulli(exp(-1)) trials
 *       Y = U + t*V;  sign bit B uniform;  start over if B = 1 and Y = 0;  Y = -Y if B = 1
 *     accept Y with probability exp(-(|Y| - s^2/t)^2 / (2 s^2))
 *
 * The publication builds its Bernoulli(exp(-x)) draws from rational arithmetic; here they are a comparison of a
 * 53-bit uniform with exp(-x) in double precision, which moves each probability by less than 2^-52: far below what
 * the chi-square tests that use this file can resolve.  Uniform bits: SplitMix64 (Steele, Lea, Flood 2014).
 */
#include <math.h>
#include <stdint.h>

static uint64_t splitmix64(uint64_t *state)
{
    uint64_t z = (*state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

static double uniform01(uint64_t *state) { return (double)(splitmix64(state) >> 11) * (1.0 / 9007199254740992.0); }

static int bernoulli_exp_minus(double x, uint64_t *state) { return uniform01(state) < exp(-x); }

/* n draws of N_Z(0, s^2), s > 0 in lattice units, into out[]; returns the number of proposals made. */
int64_t rej_dgauss_draws(double s, uint64_t seed, int64_t n, int32_t *out)
{
    uint64_t state = seed;
    const int64_t t = (int64_t)floor(s) + 1;
    int64_t proposals = 0;
    for (int64_t i = 0; i < n;) {
        int64_t u;
        do {
            u = (int64_t)(splitmix64(&state) % (uint64_t)t);
        } while (!bernoulli_exp_minus((double)u / (double)t, &state));
        int64_t v = 0;
        while (bernoulli_exp_minus(1.0, &state)) ++v;
        int64_t y = u + t * v;
        const int negative = (int)(splitmix64(&state) & 1u);
        if (negative && y == 0) continue;
        ++proposals;
        const double d = (double)y - s * s / (double)t;
        if (!bernoulli_exp_minus(d * d / (2.0 * s * s), &state)) continue;
        out[i++] = (int32_t)(negative ? -y : y);
    }
    return proposals;
}
