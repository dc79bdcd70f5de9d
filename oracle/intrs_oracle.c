/*
 * intrs_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-purpose CPU statement of what the integer randomized
 * smoothing (IntRS) PREDICT / CERTIFY loop computes, written from the paper
 * (Lin, Lou, Xiong, Shahabi: "Integer-arithmetic-only Certified Robustness for
 * Quantized Neural Networks").  It exists so that the CUDA library has
 * something independent to be compared with; it shares no code, header or
 * table with that library and nothing in the product path may call it.
 *
 * What follows the paper and what is a reading of it:
 *   - noise law               : Def. 3.3, Eq. 2 (discrete Gaussian pmf)
 *   - smoothed classifier     : Def. 3.4, Eq. 3 (argmax of vote probability)
 *   - CERTIFY                 : Algorithm 1
 *   - PREDICT                 : Algorithm 2 (Appendix C)
 *   - radius                  : Algorithm 1's return value sigma * Phi^-1(p_A)
 *   - integer-only quantile   : Theorem 3.2, steps 2-3 (lookup in the CDF of the
 *                               one-dimensional discrete Gaussian)
 *   - quantized layers        : the paper delegates them to the integer-only
 *                               scheme it cites (Sec. 1, Sec. 2 "Quantization");
 *                               the rounding, zero-point and residual rules
 *                               below are this project's reading of it.
 *   - uniform bits            : Philox4x32-10 as published by Salmon, Moraes,
 *                               Dror, Shaw (SC'11); the paper only asks for
 *                               i.i.d. draws (Algorithm 1, steps 1 and 3).
 *
 * Pins (tests/, -m "not gpu"): Philox known answers; exact-pmf chi-square,
 * symmetry, ratio and moments of the sampler; brute-force convolution written
 * a second time; requantisation against exact rationals; Clopper-Pearson and
 * normal quantile against closed forms, SciPy and the zero pattern of the
 * paper's certified-accuracy tables; PREDICT closed forms.
 * Parity unpinned: the end-to-end votes of a random network (the paper prints
 * no worked example); they are fixed only through the pinned parts above.
 *
 * Everything is sequential except orc_sample_counts, which runs independent
 * Monte-Carlo samples on OpenMP threads.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ layers */

enum { ORC_CONV2D = 0, ORC_FC = 1, ORC_GAVGPOOL = 2, ORC_MAXPOOL = 3 };

typedef struct {
    int32_t op;
    int32_t in_tensor, res_tensor;     /* res_tensor = -1: no residual add        */
    int32_t cin, cout, kh, kw, stride, pad;
    int32_t relu;
    int32_t zp_in, zp_out, zp_res;
    const int8_t *w;                   /* [cout][cin][kh][kw]                      */
    const int32_t *bias;               /* [cout]                                   */
    const int32_t *mult;               /* [cout]; pools: [1]                       */
    const int8_t *shift;               /* [cout]; pools: [1]                       */
    int32_t res_mult, res_shift;
} orc_layer;

/* ----------------------------------------------------- Philox4x32-10 (SC'11) */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {               /* Weyl key schedule between rounds         */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32-bit uniform of element e of Monte-Carlo sample j of one image.
 * Counter layout (this project's choice; the paper needs only independence):
 *   word0 = e >> 2            word1 = low 32 bits of j
 *   word2 = low 32 bits of image_id
 *   word3 = phase | (bits 32..39 of j) << 8 | (bits 32..47 of image_id) << 16
 * key = (low, high) halves of seed; the output word is e & 3.                  */
uint32_t orc_uniform_u32(uint64_t seed, uint64_t image_id, uint32_t phase,
                         uint64_t j, uint64_t e)
{
    uint32_t ctr[4], key[2], out[4];
    ctr[0] = (uint32_t)(e >> 2);
    ctr[1] = (uint32_t)(j & 0xFFFFFFFFu);
    ctr[2] = (uint32_t)(image_id & 0xFFFFFFFFu);
    ctr[3] = (phase & 0xFFu) | (uint32_t)(((j >> 32) & 0xFFu) << 8)
           | (uint32_t)(((image_id >> 32) & 0xFFFFu) << 16);
    key[0] = (uint32_t)(seed & 0xFFFFFFFFu);
    key[1] = (uint32_t)(seed >> 32);
    orc_philox4x32_10(ctr, key, out);
    return out[e & 3];
}

/* --------------------------------------- discrete Gaussian on Z (Eq. 2, mu=0) */

/* Half-width of the table for a noise std of sigma (in [0,1] pixel units):
 * the lattice is the 256 integer pixel levels, so sigma_int = 255*sigma, and
 * the support is cut at T = ceil(7*sigma_int) (mass beyond it < 3e-12).        */
int32_t orc_dgauss_halfwidth(double sigma)
{
    double sigma_int = 255.0 * sigma;
    return (int32_t)ceil(7.0 * sigma_int);
}

/* Exact pmf of Eq. 2 restricted to z = -T..T, as doubles (pmf[z+T]).           */
void orc_dgauss_pmf(double sigma, double *pmf)
{
    double sigma_int = 255.0 * sigma;
    int32_t T = orc_dgauss_halfwidth(sigma);
    double S = 0.0;
    for (int32_t z = -T; z <= T; ++z) {
        double w = exp(-(double)((int64_t)z * z) / (2.0 * sigma_int * sigma_int));
        pmf[z + T] = w;
        S += w;
    }
    for (int32_t z = -T; z <= T; ++z) pmf[z + T] /= S;
}

/* Cumulative table on a 2^-32 grid: cum[z+T] = floor(P[Z <= z] * 2^32), the
 * last entry forced to 2^32-1.  A uniform u maps to the smallest z with
 * u < cum[z+T], or to T when there is none.                                    */
void orc_dgauss_table(double sigma, uint32_t *cum)
{
    double sigma_int = 255.0 * sigma;
    int32_t T = orc_dgauss_halfwidth(sigma);
    double S = 0.0;
    for (int32_t z = -T; z <= T; ++z)
        S += exp(-(double)((int64_t)z * z) / (2.0 * sigma_int * sigma_int));
    double s = 0.0;
    for (int32_t z = -T; z <= T; ++z) {
        s += exp(-(double)((int64_t)z * z) / (2.0 * sigma_int * sigma_int));
        double v = floor(s / S * 4294967296.0);
        if (v > 4294967295.0) v = 4294967295.0;
        cum[z + T] = (uint32_t)v;
    }
    cum[2 * T] = 4294967295u;
}

/* The comparison method's noise (Sec. 4.1, "FloatRS-quant": continuous Gaussian noise added to the image, the sum
 * then quantised): on integer pixels that is delta = round(sigma_int * g), g ~ N(0, 1), whose law is
 * P[delta = z] = Phi((z + 1/2) / sigma_int) - Phi((z - 1/2) / sigma_int).  Same table form as above:
 * cum[z+T] = floor(Phi((z + 1/2) / sigma_int) * 2^32), the last entry forced to 2^32-1.                        */
void orc_rgauss_table(double sigma, uint32_t *cum)
{
    double sigma_int = 255.0 * sigma;
    int32_t T = orc_dgauss_halfwidth(sigma);
    for (int32_t z = -T; z <= T; ++z) {
        double cdf = 0.5 * erfc(-(((double)z + 0.5) / sigma_int) / sqrt(2.0));
        double v = floor(cdf * 4294967296.0);
        if (v > 4294967295.0) v = 4294967295.0;
        cum[z + T] = (uint32_t)v;
    }
    cum[2 * T] = 4294967295u;
}

/* Which noise law the sampling functions below use: 0 = the discrete Gaussian of Eq. 2 (IntRS, the default),
 * 1 = the rounded continuous Gaussian (FloatRS-quant).  Process-wide; set it before a call, not during one.     */
static int g_noise_kind = 0;
void orc_set_noise_kind(int kind) { g_noise_kind = kind ? 1 : 0; }
static void sampling_table(double sigma, uint32_t *cum)
{
    if (g_noise_kind) orc_rgauss_table(sigma, cum); else orc_dgauss_table(sigma, cum);
}

/* Inverse-CDF draw by plain linear scan of the table.                          */
int32_t orc_dgauss_from_uniform(uint32_t u, const uint32_t *cum, int32_t T)
{
    for (int32_t z = -T; z <= T; ++z)
        if (u < cum[z + T]) return z;
    return T;
}

/* Same result as the linear scan, by bisection (used where speed matters; a
 * test checks the two against each other on every table boundary).             */
static int32_t dgauss_bisect(uint32_t u, const uint32_t *cum, int32_t T)
{
    int32_t lo = 0, hi = 2 * T;        /* answer index in [lo, hi]                 */
    if (!(u < cum[hi])) return T;
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if (u < cum[mid]) hi = mid; else lo = mid + 1;
    }
    return lo - T;
}

int32_t orc_dgauss_from_uniform_fast(uint32_t u, const uint32_t *cum, int32_t T)
{
    return dgauss_bisect(u, cum, T);
}

/* n_draws noise values of sample j starting at element e0 (delta, not clamped). */
void orc_noise(uint64_t seed, uint64_t image_id, uint32_t phase, uint64_t j,
               double sigma, uint64_t e0, int64_t n_draws, int32_t *delta)
{
    int32_t T = orc_dgauss_halfwidth(sigma);
    uint32_t *cum = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(2 * T + 1));
    sampling_table(sigma, cum);
    for (int64_t i = 0; i < n_draws; ++i) {
        uint32_t u = orc_uniform_u32(seed, image_id, phase, j, e0 + (uint64_t)i);
        delta[i] = dgauss_bisect(u, cum, T);
    }
    free(cum);
}

/* Noisy, saturated network input of sample j: a0 = clamp(x + delta, 0, 255).
 * x is CHW, d = C*H*W elements (Def. 3.4: f is evaluated at x + delta; the
 * saturation to the 8-bit pixel range is taken to be part of f).              */
static void noisy_input(const uint8_t *x, int64_t d, uint64_t seed, uint64_t image_id,
                        uint32_t phase, uint64_t j, const uint32_t *cum, int32_t T,
                        int32_t *a0)
{
    for (int64_t e = 0; e < d; ++e) {
        uint32_t u = orc_uniform_u32(seed, image_id, phase, j, (uint64_t)e);
        int32_t v = (int32_t)x[e] + dgauss_bisect(u, cum, T);
        if (v < 0) v = 0;
        if (v > 255) v = 255;
        a0[e] = v;
    }
}

void orc_noisy_input(const uint8_t *x, int64_t d, uint64_t seed, uint64_t image_id,
                     uint32_t phase, uint64_t j, double sigma, uint8_t *out)
{
    int32_t T = orc_dgauss_halfwidth(sigma);
    uint32_t *cum = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(2 * T + 1));
    int32_t *a0 = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
    sampling_table(sigma, cum);
    noisy_input(x, d, seed, image_id, phase, j, cum, T, a0);
    for (int64_t e = 0; e < d; ++e) out[e] = (uint8_t)a0[e];
    free(a0);
    free(cum);
}

/* ------------------------------------------------------ integer layer rules */

/* Round-half-up right shift: floor(v / 2^n + 1/2), n >= 1.                     */
static int64_t rs(int64_t v, int n)
{
    return (v + ((int64_t)1 << (n - 1))) >> n;
}

/* Requantisation of an int32 accumulator: rs(acc*mult, 31+shift).             */
int64_t orc_requant(int32_t acc, int32_t mult, int32_t shift)
{
    return rs((int64_t)acc * (int64_t)mult, 31 + shift);
}

/* Residual branch term: rs((r - zp_res)*res_mult, 31 - res_shift).            */
int64_t orc_residual_term(int32_t r, int32_t zp_res, int32_t res_mult, int32_t res_shift)
{
    return rs((int64_t)(r - zp_res) * (int64_t)res_mult, 31 - res_shift);
}

static int32_t out_clamp(int64_t q, int relu, int32_t zp_out)
{
    int64_t lo = -128;
    if (relu && zp_out > -128) lo = zp_out;
    if (q < lo) q = lo;
    if (q > 127) q = 127;
    return (int32_t)q;
}

typedef struct { int c, h, w; } shape3;

static int layer_out_shape(const orc_layer *L, shape3 in, shape3 *out)
{
    switch (L->op) {
    case ORC_CONV2D:
    case ORC_MAXPOOL:
        if (L->stride < 1 || L->kh < 1 || L->kw < 1 || L->pad < 0) return -1;
        if (in.h + 2 * L->pad < L->kh || in.w + 2 * L->pad < L->kw) return -1;
        out->h = (in.h + 2 * L->pad - L->kh) / L->stride + 1;
        out->w = (in.w + 2 * L->pad - L->kw) / L->stride + 1;
        out->c = L->cout;
        if (L->cin != in.c) return -1;
        if (L->op == ORC_MAXPOOL && L->cout != L->cin) return -1;
        return 0;
    case ORC_FC:
        if (in.h != 1 || in.w != 1 || L->cin != in.c) return -1;
        out->c = L->cout; out->h = 1; out->w = 1;
        return 0;
    case ORC_GAVGPOOL:
        if (L->cin != in.c || L->cout != in.c) return -1;
        out->c = in.c; out->h = 1; out->w = 1;
        return 0;
    }
    return -1;
}

/* One layer on CHW int32 tensors, straight from the definitions. */
static void run_layer(const orc_layer *L, const int32_t *a, shape3 in,
                      const int32_t *res, int32_t *y, shape3 out)
{
    if (L->op == ORC_CONV2D || L->op == ORC_FC) {
        int kh = L->op == ORC_FC ? 1 : L->kh, kw = L->op == ORC_FC ? 1 : L->kw;
        int st = L->op == ORC_FC ? 1 : L->stride, pad = L->op == ORC_FC ? 0 : L->pad;
        for (int o = 0; o < out.c; ++o)
            for (int oy = 0; oy < out.h; ++oy)
                for (int ox = 0; ox < out.w; ++ox) {
                    int32_t acc = L->bias[o];
                    for (int c = 0; c < in.c; ++c)
                        for (int r = 0; r < kh; ++r)
                            for (int s = 0; s < kw; ++s) {
                                int iy = oy * st + r - pad, ix = ox * st + s - pad;
                                if (iy < 0 || iy >= in.h || ix < 0 || ix >= in.w) continue;
                                int32_t av = a[((size_t)c * in.h + iy) * in.w + ix] - L->zp_in;
                                int32_t wv = L->w[(((size_t)o * in.c + c) * kh + r) * kw + s];
                                acc += av * wv;
                            }
                    int64_t v = rs((int64_t)acc * (int64_t)L->mult[o], 31 + L->shift[o]);
                    size_t oi = ((size_t)o * out.h + oy) * out.w + ox;
                    if (res)
                        v += rs((int64_t)(res[oi] - L->zp_res) * (int64_t)L->res_mult,
                                31 - L->res_shift);
                    y[oi] = out_clamp(v + L->zp_out, L->relu, L->zp_out);
                }
    } else if (L->op == ORC_GAVGPOOL) {
        for (int c = 0; c < in.c; ++c) {
            int64_t sum = 0;
            for (int i = 0; i < in.h * in.w; ++i)
                sum += a[(size_t)c * in.h * in.w + i] - L->zp_in;
            int64_t v = rs(sum * (int64_t)L->mult[0], 31 + L->shift[0]);
            y[c] = out_clamp(v + L->zp_out, L->relu, L->zp_out);
        }
    } else { /* ORC_MAXPOOL */
        for (int c = 0; c < in.c; ++c)
            for (int oy = 0; oy < out.h; ++oy)
                for (int ox = 0; ox < out.w; ++ox) {
                    int have = 0;
                    int32_t m = 0;
                    for (int r = 0; r < L->kh; ++r)
                        for (int s = 0; s < L->kw; ++s) {
                            int iy = oy * L->stride + r - L->pad;
                            int ix = ox * L->stride + s - L->pad;
                            if (iy < 0 || iy >= in.h || ix < 0 || ix >= in.w) continue;
                            int32_t v = a[((size_t)c * in.h + iy) * in.w + ix];
                            if (!have || v > m) { m = v; have = 1; }
                        }
                    y[((size_t)c * out.h + oy) * out.w + ox] = m;
                }
    }
}

/* Shapes of all tensors (tensor 0 = input). Returns 0 or -1 on a bad list. */
static int infer_shapes(const orc_layer *layers, int n_layers, int in_c, int in_h,
                        int in_w, shape3 *shp)
{
    shp[0].c = in_c; shp[0].h = in_h; shp[0].w = in_w;
    for (int i = 0; i < n_layers; ++i) {
        const orc_layer *L = &layers[i];
        if (L->in_tensor < 0 || L->in_tensor > i) return -1;
        if (L->res_tensor > i) return -1;
        if (layer_out_shape(L, shp[L->in_tensor], &shp[i + 1])) return -1;
        if (L->res_tensor >= 0) {
            shape3 r = shp[L->res_tensor];
            if (r.c != shp[i + 1].c || r.h != shp[i + 1].h || r.w != shp[i + 1].w) return -1;
        }
    }
    return 0;
}

/* Forward pass of the base classifier f on one already-noisy input a0 (CHW,
 * values 0..255).  Writes the n_classes logits; when dump_tensor >= 0 also
 * copies that tensor (CHW, int32) to dump.  Returns 0, or -1 on a bad model.  */
int orc_forward(const orc_layer *layers, int n_layers, int in_c, int in_h, int in_w,
                const int32_t *a0, int32_t *logits, int dump_tensor, int32_t *dump)
{
    shape3 *shp = (shape3 *)malloc(sizeof(shape3) * (size_t)(n_layers + 1));
    int32_t **t = (int32_t **)calloc((size_t)(n_layers + 1), sizeof(int32_t *));
    int rc = infer_shapes(layers, n_layers, in_c, in_h, in_w, shp);
    if (rc == 0) {
        size_t n0 = (size_t)in_c * in_h * in_w;
        t[0] = (int32_t *)malloc(sizeof(int32_t) * n0);
        memcpy(t[0], a0, sizeof(int32_t) * n0);
        for (int i = 0; i < n_layers; ++i) {
            const orc_layer *L = &layers[i];
            shape3 o = shp[i + 1];
            t[i + 1] = (int32_t *)malloc(sizeof(int32_t) * (size_t)o.c * o.h * o.w);
            run_layer(L, t[L->in_tensor], shp[L->in_tensor],
                      L->res_tensor >= 0 ? t[L->res_tensor] : NULL, t[i + 1], o);
        }
        shape3 last = shp[n_layers];
        size_t nl = (size_t)last.c * last.h * last.w;
        memcpy(logits, t[n_layers], sizeof(int32_t) * nl);
        if (dump_tensor >= 0 && dump_tensor <= n_layers) {
            shape3 d = shp[dump_tensor];
            memcpy(dump, t[dump_tensor], sizeof(int32_t) * (size_t)d.c * d.h * d.w);
        }
    }
    for (int i = 0; i <= n_layers; ++i) free(t[i]);
    free(t);
    free(shp);
    return rc;
}

/* Element count of tensor k (0 = input), or -1. */
int64_t orc_tensor_size(const orc_layer *layers, int n_layers, int in_c, int in_h,
                        int in_w, int k)
{
    shape3 *shp = (shape3 *)malloc(sizeof(shape3) * (size_t)(n_layers + 1));
    int64_t r = -1;
    if (k >= 0 && k <= n_layers && infer_shapes(layers, n_layers, in_c, in_h, in_w, shp) == 0)
        r = (int64_t)shp[k].c * shp[k].h * shp[k].w;
    free(shp);
    return r;
}

/* Lowest index of the maximum (ties go to the lowest index). */
int32_t orc_argmax(const int32_t *v, int n)
{
    int32_t best = 0;
    for (int i = 1; i < n; ++i)
        if (v[i] > v[best]) best = i;
    return best;
}

/* Monte-Carlo votes (Algorithm 1 steps 1-4, Algorithm 2 steps 1-2): for
 * j = first .. first+n-1 draw the noise, run f, and count the argmax label.
 * counts[n_classes] is overwritten; logits (may be NULL) receives
 * [n][n_classes] int8.  Samples are independent and run on OpenMP threads.    */
int orc_sample_counts(const orc_layer *layers, int n_layers, int in_c, int in_h, int in_w,
                      int n_classes, const uint8_t *x, uint64_t seed, uint64_t image_id,
                      uint32_t phase, int64_t first, int64_t n, double sigma,
                      int32_t *counts, int8_t *logits)
{
    int64_t d = (int64_t)in_c * in_h * in_w;
    if (orc_tensor_size(layers, n_layers, in_c, in_h, in_w, n_layers) != n_classes) return -1;
    int32_t T = orc_dgauss_halfwidth(sigma);
    uint32_t *cum = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(2 * T + 1));
    sampling_table(sigma, cum);
    int32_t *labels = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    int bad = 0;
#pragma omp parallel
    {
        int32_t *a0 = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
        int32_t *lg = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_classes);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < n; ++i) {
            uint64_t j = (uint64_t)(first + i);
            noisy_input(x, d, seed, image_id, phase, j, cum, T, a0);
            if (orc_forward(layers, n_layers, in_c, in_h, in_w, a0, lg, -1, NULL)) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            labels[i] = orc_argmax(lg, n_classes);
            if (logits)
                for (int k = 0; k < n_classes; ++k)
                    logits[i * n_classes + k] = (int8_t)lg[k];
        }
        free(lg);
        free(a0);
    }
    for (int k = 0; k < n_classes; ++k) counts[k] = 0;
    if (!bad)
        for (int64_t i = 0; i < n; ++i) counts[labels[i]] += 1;
    free(labels);
    free(cum);
    return bad ? -1 : 0;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------- decision rules (host doubles) */

/* Upper tail of Binomial(n, p): P[X >= k], summed term by term for ascending i. */
static double binom_tail(int64_t k, int64_t n, double p)
{
    double s = 0.0;
    double lp = log(p), lq = log1p(-p);
    for (int64_t i = k; i <= n; ++i)
        s += exp(lgamma((double)n + 1.0) - lgamma((double)i + 1.0)
                 - lgamma((double)(n - i) + 1.0) + (double)i * lp + (double)(n - i) * lq);
    return s;
}

/* One-sided (1-alpha) Clopper-Pearson lower confidence bound for k successes in
 * n trials (Algorithm 1 step 5): the p at which P[X >= k] equals alpha.        */
double orc_lower_conf_bound(int64_t k, int64_t n, double alpha)
{
    if (k <= 0) return 0.0;
    if (k >= n) return exp(log(alpha) / (double)n);
    double lo = 0.0, hi = (double)k / (double)n;
    for (int it = 0; it < 64; ++it) {
        double mid = 0.5 * (lo + hi);
        if (binom_tail(k, n, mid) < alpha) lo = mid; else hi = mid;
    }
    return lo;
}

/* Standard normal quantile for p in [1/2, 1): bisection on Phi over [0, 9].    */
double orc_normal_quantile(double p)
{
    double lo = 0.0, hi = 9.0;
    for (int it = 0; it < 64; ++it) {
        double mid = 0.5 * (lo + hi);
        double phi = 0.5 * erfc(-mid / sqrt(2.0));
        if (phi < p) lo = mid; else hi = mid;
    }
    return lo;
}

/* Algorithm 1 steps 2 and 4-9 from the two count vectors.
 * Returns the class or -1 (ABSTAIN); *radius = sigma * Phi^-1(p_A) or 0.       */
int32_t orc_certify_decide(const int32_t *counts0, const int32_t *counts, int n_classes,
                           int64_t N, double sigma, double alpha, double *radius,
                           double *p_lower)
{
    int32_t cA = orc_argmax(counts0, n_classes);
    int64_t nA = counts[cA];
    double pL = orc_lower_conf_bound(nA, N, alpha);
    if (p_lower) *p_lower = pL;
    if (pL > 0.5) {
        *radius = sigma * orc_normal_quantile(pL);
        return cA;
    }
    *radius = 0.0;
    return -1;
}

/* Two-sided exact binomial test of n_a successes in m trials at p = 1/2. */
double orc_binom_pvalue_half(int64_t n_a, int64_t m)
{
    double s = 0.0;
    for (int64_t i = n_a; i <= m; ++i)
        s += exp(lgamma((double)m + 1.0) - lgamma((double)i + 1.0)
                 - lgamma((double)(m - i) + 1.0) - (double)m * log(2.0));
    double pv = 2.0 * s;
    return pv < 1.0 ? pv : 1.0;
}

/* Algorithm 2 steps 2-6: top two counts, test, class or -1. */
int32_t orc_predict_decide(const int32_t *counts, int n_classes, double alpha)
{
    int32_t cA = orc_argmax(counts, n_classes);
    int64_t nA = counts[cA], nB = -1;
    for (int k = 0; k < n_classes; ++k)
        if (k != cA && counts[k] > nB) nB = counts[k];
    if (nB < 0) nB = 0;
    double pv = orc_binom_pvalue_half(nA, nA + nB);
    return pv <= alpha ? cA : -1;
}

/* --------------------------- Theorem 3.2 steps 2-3: integer-only radius */

/* Quantile of the one-dimensional discrete Gaussian N_Z(0, sigma_int^2) by
 * lookup in its precomputed CDF table: the smallest level q with
 * cum[q+T] >= floor(p * 2^32) (p given as a 32-bit fixed-point fraction).      */
int32_t orc_dgauss_quantile_fx(uint32_t p_fx, const uint32_t *cum, int32_t T)
{
    for (int32_t z = -T; z <= T; ++z)
        if (cum[z + T] >= p_fx) return z;
    return T;
}

/* The integer-only form of the certification result (Theorem 3.2 steps 2-3; Theorem 3.1).
 * Selection and the confidence bound are Algorithm 1's (steps 2, 4, 5, 6); the radius is then read off the
 * precomputed CDF of the one-dimensional discrete Gaussian instead of the normal quantile:
 *   one-sided  (two_sided = 0): q = Phi^-1_{N_H}(p_A) in pixel levels; returns q and q^2 (squared radius);
 *   two-sided  (two_sided = 1): Theorem 3.1's radius (sigma/2)(Phi^-1(p_A^lb) - Phi^-1(p_B^ub)) with p_B^ub the
 *              Clopper-Pearson upper bound of the runner-up's count; returns d = q_A - q_B (twice the radius, so that
 *              it stays an integer) and d^2 (four times the squared radius).
 * ABSTAIN (-1, 0, 0) when p_A <= 1/2 (Algorithm 1 step 6), or two-sided when p_A^lb < p_B^ub (Theorem 3.1's premise).
 * Probabilities enter the table as floor(p * 2^32).                                                              */
int32_t orc_certify_integer_decide(const int32_t *counts0, const int32_t *counts, int n_classes, int64_t N,
                                   double sigma, double alpha, int two_sided, int32_t *out_q, int64_t *out_q2)
{
    *out_q = 0; *out_q2 = 0;
    int32_t cA = orc_argmax(counts0, n_classes);
    double pA = orc_lower_conf_bound(counts[cA], N, alpha);
    if (!(pA > 0.5)) return -1;
    int32_t T = orc_dgauss_halfwidth(sigma);
    uint32_t *cum = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(2 * T + 1));
    orc_dgauss_table(sigma, cum);
    double scaled = floor(pA * 4294967296.0);
    uint32_t pfx = scaled >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)scaled;
    int32_t qA = orc_dgauss_quantile_fx(pfx, cum, T);
    int32_t result = cA;
    if (!two_sided) {
        *out_q = qA;
        *out_q2 = (int64_t)qA * qA;
    } else {
        int64_t nB = 0;
        for (int c = 0; c < n_classes; ++c)
            if (c != cA && counts[c] > nB) nB = counts[c];
        double pB = 1.0 - orc_lower_conf_bound(N - nB, N, alpha);     /* upper bound of n_B out of N */
        if (pA < pB) {
            result = -1;
        } else {
            double sb = floor(pB * 4294967296.0);
            uint32_t pbfx = sb >= 4294967295.0 ? 0xFFFFFFFFu : (sb < 0.0 ? 0u : (uint32_t)sb);
            int32_t qB = orc_dgauss_quantile_fx(pbfx, cum, T);
            *out_q = qA - qB;
            *out_q2 = (int64_t)(qA - qB) * (qA - qB);
        }
    }
    free(cum);
    return result;
}

/* Whole CERTIFY (Algorithm 1) for one image; counts vectors may be NULL.       */
int orc_certify(const orc_layer *layers, int n_layers, int in_c, int in_h, int in_w,
                int n_classes, const uint8_t *x, uint64_t seed, uint64_t image_id,
                int64_t N0, int64_t N, double sigma, double alpha,
                int32_t *out_class, double *out_radius, int32_t *out_counts0,
                int32_t *out_counts)
{
    int32_t *c0 = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_classes);
    int32_t *c1 = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_classes);
    int rc = orc_sample_counts(layers, n_layers, in_c, in_h, in_w, n_classes, x, seed,
                               image_id, 0, 0, N0, sigma, c0, NULL);
    if (!rc)
        rc = orc_sample_counts(layers, n_layers, in_c, in_h, in_w, n_classes, x, seed,
                               image_id, 1, 0, N, sigma, c1, NULL);
    if (!rc) {
        *out_class = orc_certify_decide(c0, c1, n_classes, N, sigma, alpha, out_radius, NULL);
        if (out_counts0) memcpy(out_counts0, c0, sizeof(int32_t) * (size_t)n_classes);
        if (out_counts) memcpy(out_counts, c1, sizeof(int32_t) * (size_t)n_classes);
    }
    free(c0);
    free(c1);
    return rc;
}

/* Whole PREDICT (Algorithm 2) for one image. */
int orc_predict(const orc_layer *layers, int n_layers, int in_c, int in_h, int in_w,
                int n_classes, const uint8_t *x, uint64_t seed, uint64_t image_id,
                int64_t N, double sigma, double alpha, int32_t *out_class,
                int32_t *out_counts)
{
    int32_t *c = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_classes);
    int rc = orc_sample_counts(layers, n_layers, in_c, in_h, in_w, n_classes, x, seed,
                               image_id, 2, 0, N, sigma, c, NULL);
    if (!rc) {
        *out_class = orc_predict_decide(c, n_classes, alpha);
        if (out_counts) memcpy(out_counts, c, sizeof(int32_t) * (size_t)n_classes);
    }
    free(c);
    return rc;
}
