/*
 * tq_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-threaded CPU statement of the truncated-quantization gradient
 * compressor of "Improved Quantization Strategies for Managing Heavy-tailed Gradients in
 * Distributed Learning" (Yan, Li, Xiao, Hou, Song), written from the paper so that the
 * CUDA library can be compared with it.  It shares no code, header, table or constant
 * generator with the CUDA library, and the library never calls it.  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * Build:  gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -shared -fPIC tq_oracle.c -lm
 * (-ffp-contract=off matters: the code decisions below are taken in fp32 with one
 * rounding per operation and no fused multiply-add.)
 *
 * What the paper fixes, and where:
 *   truncation T_alpha ........................ Section 3.1, truncation equation
 *   stochastic quantizer Q on a codebook ...... Section 3.1, quantizer equation; Lemma 1
 *   density <-> codebook, integral = s ........ Section 3.1 (paragraph after Lemma 1)
 *   uniform codebook .......................... Section 4.1, first paragraph
 *   power-law tail model, rho, g_min .......... Section 4.1, power-law definition + tail model
 *   E_TQ(alpha), uniform ...................... Section 4.1, error equation
 *   alpha, uniform (boxed) / alpha' ........... Section 4.1, boxed equation / text after Theorem 1
 *   Theorem 1 error at the optimum ............ Section 4.1, Theorem 1; Appendix proof of Theorem 1
 *   lambda_s proportional to p^(1/3) (boxed) .. Section 4.2, boxed density
 *   Q_N(alpha), alpha non-uniform (boxed) ..... Section 4.2
 *   gamma maximum-likelihood estimate ......... Section 5, experimental setting
 *   BiScaled density, Q_B, alpha (boxed) ...... Appendix, "Truncated BiScaled Quantization"
 *   server aggregation ........................ Algorithm 1, server step; Lemma 2 (w_i = 1/N)
 *
 * What the paper leaves open is fixed here (one reading each, listed for the reader):
 *   R1  num_levels L = 2^b quantization points, s = L - 1 intervals (Section 3.1).
 *   R2  rho is the ONE-SIDED tail mass, rho = P(g > g_min) = P(|g| > g_min) / 2: only this
 *       reproduces the second term of the uniform error equation from Lemma 2's bias term.
 *   R3  g_min is given by the caller, or kappa * mean|g|.
 *   R4  the MLE pools both signs: it runs over |g_j| > g_min.
 *   R5  the alpha equations are used for every gamma > 2 (they only need the first tail
 *       moment); the closed-form ERROR expressions need gamma > 3.
 *   R6  below g_min the model density is flat, p = (1 - 2 rho) / (2 g_min).
 *   R7  levels follow from the density by companding: integral_{-alpha}^{l_k} lambda_s = k.
 *   R8  "alternating iterations": start at alpha', iterate the boxed equation with the
 *       model Q_U / Q_N, at most 10000 times, stop at relative change <= 1e-12; the result
 *       is clamped to [g_min, max|g|].
 *   R9  randomness: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), key = the 64-bit
 *       seed, counter = (j >> 3 as two words, worker, 0); element j takes 16-bit slot j & 7 of the
 *       128 output bits (slot q = low/high half (q & 1) of output word q >> 1).
 *   R10 rounding decision in fp32: T = rint(p * 2^16), round up iff r < T.  P(up) is p
 *       rounded to the nearest multiple of 2^-16, so the quantizer is unbiased to
 *       |Delta_k| * 2^-17 per element and exactly unbiased on average over p.
 *   R11 the inverse widths are rounded UP to fp32, so a value on the top level l_s gets
 *       probability >= 1 and always receives code s (Section 3.1: |g| > alpha maps to
 *       sgn(g) alpha, which is a codebook point).
 *   R12 wire format: dense LSB-first bit stream over little-endian 32-bit words, pad zero.
 *   R16 the no-truncation baselines of Section 5 (QSGD, NQSGD) are the same quantizers with
 *       alpha = max|g| (alpha rule MAXABS), so that the truncation operator is the identity.
 *   R17 truncated BiScaled quantizer (Appendix): k* = argmin_k Q_B(alpha, k) is found by a scan of
 *       k = j/64 followed by 60 golden-section steps in the bracketing pair of cells; alpha iterates the
 *       boxed BiScaled equation as in R8 with k* recomputed at every step; s_alpha, s_beta are real
 *       numbers (the Appendix's formulas), so the levels come from the two-piece density by R7.
 *   R18 the server's model update (Algorithm 1, last step) is the momentum SGD with weight decay of
 *       Section 5: g += wd*theta; m = mu*m + g; theta -= lr*m; fp32, each operation rounded once.
 *   R13 aggregation: fp32 adds in worker order, then one IEEE division by N; with
 *       weights, each product w_i * v_i is rounded, then added, no division.
 *   R14 non-finite gradients: counted by the statistics and left out of every sum; the quantizer
 *       sends NaN to -alpha (code 0) and +-Inf to +-alpha (fmaxf / fminf semantics).
 *   R15 uniform index: x = (t + alpha) * inv_step in fp32, two roundings; k = min(floor x, s-1).
 *   R19 one-pass statistics: the automatic threshold kappa * mean|g| is rounded DOWN to a power of
 *       two (0, i.e. no tail, below the smallest normal number): orc_pow2_floor, orc_stats_pow2.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#define ORC_MAX_LEVELS 16

enum { ORC_OK = 0, ORC_ERR_ARG = -1, ORC_ERR_DOMAIN = -2, ORC_ERR_LEVELS = -5 };
enum { ORC_UNIFORM = 0, ORC_NONUNIFORM = 1, ORC_BISCALED = 2 };
enum { ORC_ALPHA_CLOSED = 0, ORC_ALPHA_FIXED_POINT = 1, ORC_ALPHA_USER = 2, ORC_ALPHA_MAXABS = 3 };
enum { ORC_FLAG_ALPHA_CAPPED = 1, ORC_FLAG_ALPHA_AT_GMIN = 2, ORC_FLAG_GAMMA_FROM_MLE = 4 };

/* ------------------------------------------------------------------------------------ */
/* R9: Philox4x32-10.  One round multiplies counter words 0 and 2 by two fixed odd       */
/* constants, keeps both halves of each 64-bit product, and mixes the high halves with   */
/* the other two counter words and the round key; the key advances by a Weyl sequence.  */
/* ------------------------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* R9: the 16 random bits of element j of one worker. */
uint32_t orc_rand16(uint64_t seed, uint32_t worker, uint64_t j)
{
    uint64_t block = j >> 3;
    uint32_t ctr[4] = { (uint32_t)block, (uint32_t)(block >> 32), worker, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    uint32_t slot = (uint32_t)(j & 7u);
    uint32_t word = out[slot >> 1];
    return (slot & 1u) ? (word >> 16) : (word & 0xFFFFu);
}

/* bf16 -> fp32: the 16 stored bits are the high half of the fp32 pattern (exact). */
void orc_bf16_to_f32(const uint16_t *in, uint64_t n, float *out)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t bits = (uint32_t)in[i] << 16;
        memcpy(&out[i], &bits, 4);
    }
}

/* ------------------------------------------------------------------------------------ */
/* Statistics of one worker's gradient (Section 5: gamma MLE; Section 4.1: rho, g_min). */
/* ------------------------------------------------------------------------------------ */
typedef struct {
    uint64_t d, n_tail, n_nonfinite;
    double sum_abs, sum_sq, sum_log_tail;
    float max_abs, g_min;
} orc_stats_t;

/* g_min_in > 0: use it.  Otherwise g_min = (float)(kappa * mean|g|) (R3). */
int orc_stats(const float *g, uint64_t d, float g_min_in, double kappa, orc_stats_t *st)
{
    if (!g && d) return ORC_ERR_ARG;
    memset(st, 0, sizeof *st);
    st->d = d;
    double sum_abs = 0.0, sum_sq = 0.0;
    float max_abs = 0.0f;
    uint64_t bad = 0;
    for (uint64_t j = 0; j < d; ++j) {
        float x = g[j];
        if (!isfinite(x)) { ++bad; continue; }
        float a = fabsf(x);
        sum_abs += (double)a;
        sum_sq += (double)a * (double)a;
        if (a > max_abs) max_abs = a;
    }
    st->sum_abs = sum_abs; st->sum_sq = sum_sq; st->max_abs = max_abs; st->n_nonfinite = bad;
    float g_min = g_min_in;
    if (!(g_min_in > 0.0f))
        g_min = d ? (float)(kappa * sum_abs / (double)d) : 0.0f;
    st->g_min = g_min;
    uint64_t n_tail = 0;
    double sum_log = 0.0;
    if (g_min > 0.0f) {
        for (uint64_t j = 0; j < d; ++j) {
            float x = g[j];
            if (!isfinite(x)) continue;
            float a = fabsf(x);
            if (a > g_min) {                       /* R4 */
                ++n_tail;
                sum_log += log((double)a / (double)g_min);
            }
        }
    }
    st->n_tail = n_tail; st->sum_log_tail = sum_log;
    return ORC_OK;
}

/* R19: the power-of-two threshold rule.  The largest power of two not above x, written with the
 * C library's frexp / ldexp; 0 below the smallest normal float (no tail), Inf for Inf.
 * The statistics under this rule are orc_stats called with g_min = orc_pow2_floor(kappa * mean|g|),
 * the mean taken from a first orc_stats call (see stats_pow2 in the Python wrapper). */
float orc_pow2_floor(float x)
{
    if (!(x >= FLT_MIN)) return 0.0f;
    if (isinf(x)) return x;
    int e;
    (void)frexpf(x, &e);            /* x = m * 2^e, 0.5 <= m < 1 */
    return ldexpf(0.5f, e);
}

/* ------------------------------------------------------------------------------------ */
/* The density model (Section 4.1 tail model + R6) and what follows from it.            */
/* ------------------------------------------------------------------------------------ */
typedef struct { double g_min, rho, gamma; } orc_model_t;

/* p(g): flat body below g_min, power-law tail above. */
double orc_model_pdf(const orc_model_t *m, double g)
{
    double a = fabs(g);
    if (a <= m->g_min) return (1.0 - 2.0 * m->rho) / (2.0 * m->g_min);
    return m->rho * (m->gamma - 1.0) * pow(m->g_min, m->gamma - 1.0) * pow(a, -m->gamma);
}

/* Q_U(alpha) = integral_{-alpha}^{alpha} p  (Section 4.1, definition under the error equation). */
double orc_model_QU(const orc_model_t *m, double alpha)
{
    if (alpha <= m->g_min) return (1.0 - 2.0 * m->rho) * alpha / m->g_min;
    return 1.0 - 2.0 * m->rho * pow(alpha / m->g_min, 1.0 - m->gamma);
}

/* H(x) = integral_0^x p^(1/3), x >= 0: the (unnormalised) compander of the boxed density. */
double orc_model_H(const orc_model_t *m, double x)
{
    double cb = cbrt((1.0 - 2.0 * m->rho) / (2.0 * m->g_min));
    if (x <= m->g_min) return cb * x;
    double A = cbrt(m->rho * (m->gamma - 1.0)) * pow(m->g_min, (m->gamma - 1.0) / 3.0);
    double beta = 1.0 - m->gamma / 3.0;
    if (beta == 0.0) return cb * m->g_min + A * log(x / m->g_min);
    return cb * m->g_min + A * (pow(x, beta) - pow(m->g_min, beta)) / beta;
}

/* Inverse of H on tau >= 0. */
double orc_model_Hinv(const orc_model_t *m, double tau)
{
    double cb = cbrt((1.0 - 2.0 * m->rho) / (2.0 * m->g_min));
    double body = cb * m->g_min;
    if (tau <= body) return tau / cb;
    double A = cbrt(m->rho * (m->gamma - 1.0)) * pow(m->g_min, (m->gamma - 1.0) / 3.0);
    double beta = 1.0 - m->gamma / 3.0;
    if (beta == 0.0) return m->g_min * exp((tau - body) / A);
    return pow(pow(m->g_min, beta) + beta * (tau - body) / A, 1.0 / beta);
}

/* Q_N(alpha) = [ integral_{-alpha}^{alpha} p^(1/3) (1/(2 alpha))^(2/3) ]^3 = 2 H(alpha)^3 / alpha^2. */
double orc_model_QN(const orc_model_t *m, double alpha)
{
    double h = orc_model_H(m, alpha);
    return 2.0 * h * h * h / (alpha * alpha);
}

/* Appendix: Q_B(alpha, k) = [ (2 int_{k alpha}^{alpha} p)^(1/3) (1-k)^(2/3) + (2 int_0^{k alpha} p)^(1/3) k^(2/3) ]^3 */
double orc_model_QB(const orc_model_t *m, double alpha, double k)
{
    double inner = orc_model_QU(m, k * alpha);               /* 2 int_0^{k alpha} p */
    double outer = orc_model_QU(m, alpha) - inner;           /* 2 int_{k alpha}^{alpha} p */
    if (outer < 0.0) outer = 0.0;
    double t = cbrt(outer) * pow(1.0 - k, 2.0 / 3.0) + cbrt(inner) * pow(k, 2.0 / 3.0);
    return t * t * t;
}

/* R17: k* = argmin_k Q_B(alpha, k) on [0, 1]. */
double orc_biscaled_kstar(const orc_model_t *m, double alpha)
{
    int best = 0;
    double best_q = orc_model_QB(m, alpha, 0.0);
    for (int j = 1; j <= 64; ++j) {
        double q = orc_model_QB(m, alpha, (double)j / 64.0);
        if (q < best_q) { best_q = q; best = j; }
    }
    double lo = (best > 0 ? best - 1 : 0) / 64.0, hi = (best < 64 ? best + 1 : 64) / 64.0;
    const double r = 0.6180339887498949;                     /* (sqrt 5 - 1) / 2 */
    double x1 = hi - r * (hi - lo), x2 = lo + r * (hi - lo);
    double f1 = orc_model_QB(m, alpha, x1), f2 = orc_model_QB(m, alpha, x2);
    for (int it = 0; it < 60; ++it) {
        if (f1 <= f2) { hi = x2; x2 = x1; f2 = f1; x1 = hi - r * (hi - lo); f1 = orc_model_QB(m, alpha, x1); }
        else          { lo = x1; x1 = x2; f1 = f2; x2 = lo + r * (hi - lo); f2 = orc_model_QB(m, alpha, x2); }
    }
    return 0.5 * (lo + hi);
}

/* The boxed BiScaled density: lambda_in on |g| <= k* alpha, lambda_out on k* alpha < |g| <= alpha. */
void orc_biscaled_density(const orc_model_t *m, double alpha, double s, double *k_out, double *lam_in, double *lam_out)
{
    double k = orc_biscaled_kstar(m, alpha);
    double beta = k * alpha;
    double p1 = orc_model_QU(m, beta) / (2.0 * beta);                              /* mean density on [0, beta] */
    double p2 = (orc_model_QU(m, alpha) - orc_model_QU(m, beta)) / (2.0 * (alpha - beta));
    double c1 = cbrt(p1), c2 = cbrt(p2);
    double denom = 2.0 * c2 * (1.0 - k) * alpha + 2.0 * c1 * k * alpha;
    *k_out = k; *lam_in = c1 * s / denom; *lam_out = c2 * s / denom;
}

/* Truncation-bias term of the error equations, per element and per 1/N:
 * 4 rho g_min^(gamma-1) alpha^(3-gamma) / ((gamma-2)(gamma-3)); needs gamma > 3, alpha >= g_min. */
double orc_truncation_bias(const orc_model_t *m, double alpha)
{
    return 4.0 * m->rho * pow(m->g_min, m->gamma - 1.0) * pow(alpha, 3.0 - m->gamma)
           / ((m->gamma - 2.0) * (m->gamma - 3.0));
}

/* E_TQ(alpha) * N / d for the uniform quantizer (Section 4.1 error equation). */
double orc_etq_uniform(const orc_model_t *m, double alpha, double s)
{
    return orc_model_QU(m, alpha) * alpha * alpha / (s * s) + orc_truncation_bias(m, alpha);
}

/* E_TQ(alpha) * N / d for the p^(1/3) density (Section 4.2 error equation with the boxed density
 * substituted: (1/4) integral p / lambda^2 = Q_N alpha^2 / s^2). */
double orc_etq_nonuniform(const orc_model_t *m, double alpha, double s)
{
    return orc_model_QN(m, alpha) * alpha * alpha / (s * s) + orc_truncation_bias(m, alpha);
}

/* E_TQ(alpha, k*) * N / d for the BiScaled density (Appendix error equation). */
double orc_etq_biscaled(const orc_model_t *m, double alpha, double s)
{
    return orc_model_QB(m, alpha, orc_biscaled_kstar(m, alpha)) * alpha * alpha / (s * s) + orc_truncation_bias(m, alpha);
}

/* Theorems 1 and 2: the error term at the optimum, given Q = Q_U(alpha*) or Q_N(alpha*). */
double orc_etq_theorem(const orc_model_t *m, double Q, double s)
{
    double gm1 = m->gamma - 1.0;
    return gm1 * pow(Q, (m->gamma - 3.0) / gm1) * m->g_min * m->g_min * pow(2.0 * m->rho, 2.0 / gm1)
           * pow(s, (6.0 - 2.0 * m->gamma) / gm1)
           / ((m->gamma - 3.0) * pow(m->gamma - 2.0, 2.0 / gm1));
}

/* alpha' (text after Theorem 1): the boxed equation with Q = 1. */
double orc_alpha_prime(const orc_model_t *m, double s)
{
    return m->g_min * pow(2.0 * m->rho * s * s / (m->gamma - 2.0), 1.0 / (m->gamma - 1.0));
}

/* One application of the boxed equation's right-hand side. */
static double alpha_map(const orc_model_t *m, double s, int mode, double alpha)
{
    double Q = (mode == ORC_UNIFORM) ? orc_model_QU(m, alpha)
             : (mode == ORC_NONUNIFORM) ? orc_model_QN(m, alpha)
             : orc_model_QB(m, alpha, orc_biscaled_kstar(m, alpha));
    return m->g_min * pow(2.0 * m->rho * s * s / ((m->gamma - 2.0) * Q), 1.0 / (m->gamma - 1.0));
}

/* R8: the alternating iteration.  Returns alpha; *iters and *capped are reported. */
double orc_alpha_fixed_point(const orc_model_t *m, double s, int mode, double alpha_cap,
                             int *iters, int *capped)
{
    double alpha = orc_alpha_prime(m, s);
    int it = 0, cap = 0;
    for (; it < 10000; ++it) {
        if (alpha_cap > 0.0 && alpha > alpha_cap) { cap = 1; break; }
        double next = alpha_map(m, s, mode, alpha);
        double change = fabs(next - alpha);
        alpha = next;
        if (change <= 1e-12 * fabs(next)) { ++it; break; }
    }
    if (alpha_cap > 0.0 && alpha > alpha_cap) cap = 1;
    if (iters) *iters = it;
    if (capped) *capped = cap;
    return alpha;
}

/* smallest fp32 that is >= v (v > 0 finite) */
static float round_up_f32(double v)
{
    float f = (float)v;
    if ((double)f < v) f = nextafterf(f, INFINITY);
    return f;
}

typedef struct {
    uint32_t bits, num_levels, mode, flags;
    float alpha, inv_step, gamma, g_min, rho;
    int32_t iterations;
    float levels[ORC_MAX_LEVELS];
    float inv_width[ORC_MAX_LEVELS];
} orc_params_t;

/* R11: inverse widths and inverse step, rounded up; alpha = l_s. */
static int finish_table(orc_params_t *p, uint32_t s)
{
    float alpha_f = p->levels[s];
    for (uint32_t k = 0; k < s; ++k) {
        if (!(p->levels[k + 1] > p->levels[k])) return ORC_ERR_LEVELS;
        float width = (float)((double)p->levels[k + 1] - (double)p->levels[k]);
        p->inv_width[k] = round_up_f32(1.0 / (double)width);
        if (!isfinite(p->inv_width[k])) return ORC_ERR_LEVELS;
    }
    p->inv_step = round_up_f32((double)s / (double)(2.0f * alpha_f));
    if (!isfinite(p->inv_step)) return ORC_ERR_LEVELS;
    p->alpha = alpha_f;
    return ORC_OK;
}

/* Fill levels/inverse widths/inv_step for a given fp32 alpha (R7, R11). */
int orc_build_table(const orc_model_t *m, uint32_t num_levels, int mode, float alpha_f, orc_params_t *p)
{
    uint32_t s = num_levels - 1;
    double a = (double)alpha_f;
    if (!(alpha_f > 0.0f) || !isfinite(2.0f * alpha_f)) return ORC_ERR_DOMAIN;
    for (int k = 0; k < ORC_MAX_LEVELS; ++k) { p->levels[k] = 0.0f; p->inv_width[k] = 0.0f; }
    if (mode == ORC_UNIFORM) {
        /* Section 4.1: l_k = -alpha + k * 2 alpha / s */
        for (uint32_t k = 0; k <= s; ++k)
            p->levels[k] = (float)(-a + (double)k * (2.0 * a / (double)s));
    } else if (mode == ORC_BISCALED) {
        /* R17 + R7: cumulative density from the centre reaches k - s/2 at level k */
        double kk, lam_in, lam_out;
        orc_biscaled_density(m, a, (double)s, &kk, &lam_in, &lam_out);
        double beta = kk * a;
        for (uint32_t k = 0; k <= s; ++k) {
            if (2 * k < s) continue;
            double c = (double)k - 0.5 * (double)s;
            double x = (c <= lam_in * beta) ? c / lam_in : beta + (c - lam_in * beta) / lam_out;
            float l = (float)x;
            p->levels[k] = l;
            p->levels[s - k] = -l;
        }
    } else {
        /* R7: H(l_k) = (2k/s - 1) H(alpha); upper half computed, lower half mirrored */
        double Ha = orc_model_H(m, a);
        for (uint32_t k = 0; k <= s; ++k) {
            if (2 * k < s) continue;
            double tau = (2.0 * (double)k / (double)s - 1.0) * Ha;
            float l = (float)orc_model_Hinv(m, tau);
            p->levels[k] = l;
            p->levels[s - k] = -l;
        }
    }
    p->levels[0] = -alpha_f;
    p->levels[s] = alpha_f;
    return finish_table(p, s);
}

/* Params for a caller-supplied codebook l_0 < ... < l_s with l_0 = -l_s (no density model). */
int orc_table_from_levels(const float *levels, uint32_t num_levels, int mode, orc_params_t *p)
{
    memset(p, 0, sizeof *p);
    uint32_t bits = 0;
    while (bits < 5 && (1u << bits) != num_levels) ++bits;
    if (bits < 1 || bits > 4) return ORC_ERR_ARG;
    p->bits = bits; p->num_levels = num_levels; p->mode = (uint32_t)mode;
    for (uint32_t k = 0; k < num_levels; ++k) p->levels[k] = levels[k];
    if (!(levels[num_levels - 1] > 0.0f) || levels[0] != -levels[num_levels - 1]) return ORC_ERR_DOMAIN;
    return finish_table(p, num_levels - 1);
}

/* Section 4 as a whole: statistics -> (alpha, codebook).  gamma = NaN asks for the MLE. */
int orc_params(const orc_stats_t *st, uint32_t num_levels, int mode, double gamma,
               int alpha_rule, double alpha_user, orc_params_t *p)
{
    memset(p, 0, sizeof *p);
    uint32_t bits = 0;
    while (bits < 5 && (1u << bits) != num_levels) ++bits;
    if (bits < 1 || bits > 4) return ORC_ERR_ARG;
    if (mode != ORC_UNIFORM && mode != ORC_NONUNIFORM && mode != ORC_BISCALED) return ORC_ERR_ARG;
    p->bits = bits; p->num_levels = num_levels; p->mode = (uint32_t)mode;
    double s = (double)(num_levels - 1);

    if (isnan(gamma)) {                            /* Section 5 MLE (R4) */
        if (!(st->n_tail > 0) || !(st->sum_log_tail > 0.0)) return ORC_ERR_DOMAIN;
        gamma = 1.0 + (double)st->n_tail / st->sum_log_tail;
        p->flags |= ORC_FLAG_GAMMA_FROM_MLE;
    }
    if (!(gamma > 2.0) || !isfinite(gamma)) return ORC_ERR_DOMAIN;     /* R5 */
    if (!(st->g_min > 0.0f) || !isfinite(st->g_min) || st->d == 0) return ORC_ERR_DOMAIN;
    double rho = (double)st->n_tail / (2.0 * (double)st->d);          /* R2 */
    if (!(rho > 0.0) || !(rho < 0.5)) return ORC_ERR_DOMAIN;
    orc_model_t m = { (double)st->g_min, rho, gamma };
    p->gamma = (float)gamma; p->g_min = st->g_min; p->rho = (float)rho;

    double alpha;
    if (alpha_rule == ORC_ALPHA_USER) {
        if (!(alpha_user > 0.0) || !isfinite(alpha_user)) return ORC_ERR_DOMAIN;
        alpha = alpha_user;
    } else if (alpha_rule == ORC_ALPHA_MAXABS) {
        /* Section 5 baselines QSGD / NQSGD: quantization without truncation, the range is max|g| */
        if (!(st->max_abs > 0.0f)) return ORC_ERR_DOMAIN;
        alpha = (double)st->max_abs;
    } else {
        double cap = (double)st->max_abs;
        int capped = 0, iters = 0;
        if (alpha_rule == ORC_ALPHA_CLOSED) alpha = orc_alpha_prime(&m, s);
        else if (alpha_rule == ORC_ALPHA_FIXED_POINT)
            alpha = orc_alpha_fixed_point(&m, s, mode, cap, &iters, &capped);
        else return ORC_ERR_ARG;
        p->iterations = iters;
        if (!(alpha == alpha)) return ORC_ERR_DOMAIN;
        if (alpha < m.g_min) { alpha = m.g_min; p->flags |= ORC_FLAG_ALPHA_AT_GMIN; }
        if (cap > 0.0 && alpha > cap) { alpha = cap; p->flags |= ORC_FLAG_ALPHA_CAPPED; }
    }
    return orc_build_table(&m, num_levels, mode, (float)alpha, p);
}

/* ------------------------------------------------------------------------------------ */
/* Per-element compressor: Section 3.1 truncation + quantizer, decisions in fp32.       */
/* ------------------------------------------------------------------------------------ */

/* T_alpha.  fmaxf/fminf return the non-NaN operand, so NaN -> -alpha; +-Inf -> +-alpha. */
static float truncate_alpha(float g, float alpha)
{
    return fminf(fmaxf(g, -alpha), alpha);
}

/* Interval index k (value lies in [l_k, l_{k+1}]) and round-up probability p_r for a
 * truncated value t.  Returns k, writes p. */
static uint32_t interval_and_prob(const orc_params_t *q, float t, float *p_out)
{
    uint32_t s = q->num_levels - 1;
    uint32_t k;
    float p;
    if (q->mode == ORC_UNIFORM) {
        float shifted = t + q->alpha;              /* one rounding */
        float x = shifted * q->inv_step;           /* one rounding */
        k = (uint32_t)x;                           /* truncation; x >= 0 */
        if (k > s - 1) k = s - 1;
        p = x - (float)k;                          /* exact */
    } else {
        k = 0;
        for (uint32_t j = 1; j + 1 <= s; ++j)      /* largest j <= s-1 with l_j <= t */
            if (q->levels[j] <= t) k = j;
        float off = t - q->levels[k];              /* one rounding */
        p = off * q->inv_width[k];                 /* one rounding */
    }
    *p_out = p;
    return k;
}

/* R10: integer threshold of the rounding decision. */
static uint32_t up_threshold(float p)
{
    float scaled = p * 65536.0f;                   /* exact: power-of-two scaling */
    return (uint32_t)(int32_t)rintf(scaled);       /* ties to even (default rounding mode) */
}

/* Code of one element, given its 16 random bits. */
uint32_t orc_code_from_bits(const orc_params_t *q, float g, uint32_t r16)
{
    float p;
    float t = truncate_alpha(g, q->alpha);
    uint32_t k = interval_and_prob(q, t, &p);
    return k + ((r16 < up_threshold(p)) ? 1u : 0u);
}

/* Code of element j of a worker (random bits from R9). */
uint32_t orc_code_at(const orc_params_t *q, float g, uint64_t seed, uint32_t worker, uint64_t j)
{
    return orc_code_from_bits(q, g, orc_rand16(seed, worker, j));
}

/* For the pins: interval k, probability p and threshold T of a value. */
void orc_decision(const orc_params_t *q, float g, float *t_out, uint32_t *k_out, float *p_out, uint32_t *T_out)
{
    float p;
    float t = truncate_alpha(g, q->alpha);
    uint32_t k = interval_and_prob(q, t, &p);
    *t_out = t; *k_out = k; *p_out = p; *T_out = up_threshold(p);
}

/* All codes of one worker, one byte each. */
void orc_quantize(const float *g, uint64_t d, const orc_params_t *q, uint64_t seed, uint32_t worker,
                  uint8_t *codes)
{
    for (uint64_t j = 0; j < d; ++j)
        codes[j] = (uint8_t)orc_code_at(q, g[j], seed, worker, j);
}

/* Codes of the n elements j0 .. j0+n-1 of a longer vector (g points at element j0): the random
 * bits depend on the absolute index, so a window of a large gradient can be checked on its own. */
void orc_quantize_window(const float *g, uint64_t n, uint64_t j0, const orc_params_t *q, uint64_t seed,
                         uint32_t worker, uint8_t *codes)
{
    for (uint64_t i = 0; i < n; ++i)
        codes[i] = (uint8_t)orc_code_at(q, g[i], seed, worker, j0 + i);
}

/* R12: words needed for d codes of `bits` bits, rounded up to a multiple of 4 words. */
uint64_t orc_packed_words(uint64_t d, uint32_t bits)
{
    uint64_t raw = (d * (uint64_t)bits + 31u) / 32u;
    return (raw + 3u) / 4u * 4u;
}

/* R12: code j occupies stream bits [j*bits, (j+1)*bits); bit i of the stream is bit (i & 31)
 * of word (i >> 5).  All `words` words are written (unused bits zero). */
void orc_pack(const uint8_t *codes, uint64_t d, uint32_t bits, uint32_t *packed, uint64_t words)
{
    for (uint64_t w = 0; w < words; ++w) packed[w] = 0u;
    for (uint64_t j = 0; j < d; ++j) {
        uint64_t pos = j * (uint64_t)bits;
        for (uint32_t i = 0; i < bits; ++i) {
            uint64_t bit = pos + i;
            if ((codes[j] >> i) & 1u) packed[bit >> 5] |= (uint32_t)1u << (bit & 31u);
        }
    }
}

void orc_unpack(const uint32_t *packed, uint64_t d, uint32_t bits, uint8_t *codes)
{
    for (uint64_t j = 0; j < d; ++j) {
        uint64_t pos = j * (uint64_t)bits;
        uint32_t c = 0;
        for (uint32_t i = 0; i < bits; ++i) {
            uint64_t bit = pos + i;
            c |= ((packed[bit >> 5] >> (bit & 31u)) & 1u) << i;
        }
        codes[j] = (uint8_t)c;
    }
}

/* Client side of Algorithm 1 for one worker: quantize every element and pack. */
int orc_compress(const float *g, uint64_t d, const orc_params_t *q, uint64_t seed, uint32_t worker,
                 uint32_t *packed, uint64_t words, uint8_t *scratch_codes)
{
    if (words < orc_packed_words(d, q->bits)) return ORC_ERR_ARG;
    orc_quantize(g, d, q, seed, worker, scratch_codes);
    orc_pack(scratch_codes, d, q->bits, packed, words);
    return ORC_OK;
}

/* Server side of Algorithm 1 (R13).  packed is [n_workers][stride_words]; params one per worker. */
int orc_decompress_aggregate(const uint32_t *packed, uint64_t stride_words, uint32_t n_workers,
                             uint64_t d, const orc_params_t *params, const float *weights, float *out)
{
    if (n_workers == 0) return ORC_ERR_ARG;
    for (uint32_t i = 1; i < n_workers; ++i)
        if (params[i].bits != params[0].bits) return ORC_ERR_ARG;
    uint32_t bits = params[0].bits;
    for (uint64_t j = 0; j < d; ++j) {
        float acc = 0.0f;
        for (uint32_t i = 0; i < n_workers; ++i) {
            const uint32_t *pw = packed + (uint64_t)i * stride_words;
            uint64_t pos = j * (uint64_t)bits;
            uint32_t c = 0;
            for (uint32_t b = 0; b < bits; ++b) {
                uint64_t bit = pos + b;
                c |= ((pw[bit >> 5] >> (bit & 31u)) & 1u) << b;
            }
            float v = params[i].levels[c];
            if (weights) {
                float wv = weights[i] * v;         /* rounded product */
                acc = acc + wv;
            } else {
                acc = acc + v;
            }
        }
        out[j] = weights ? acc : acc / (float)n_workers;
    }
    return ORC_OK;
}

/* Server side of Algorithm 1 including the model update (last step of the round), with the optimiser of
 * the paper's experiments (Section 5: momentum SGD with weight decay).  R18: fp32, one rounding per
 * operation: g = aggregate (R13); g += wd * theta (if wd != 0); m = mu * m + g (if a momentum buffer is
 * given); theta -= lr * (m or g). */
int orc_decompress_aggregate_apply(const uint32_t *packed, uint64_t stride_words, uint32_t n_workers,
                                   uint64_t d, const orc_params_t *params, const float *weights,
                                   float *theta, float *momentum_buf, float lr, float mu, float wd, float *scratch)
{
    int rc = orc_decompress_aggregate(packed, stride_words, n_workers, d, params, weights, scratch);
    if (rc != ORC_OK) return rc;
    for (uint64_t j = 0; j < d; ++j) {
        float g = scratch[j];
        if (wd != 0.0f) {
            float decay = wd * theta[j];
            g = g + decay;
        }
        if (momentum_buf) {
            float carried = mu * momentum_buf[j];
            float m = carried + g;
            momentum_buf[j] = m;
            g = m;
        }
        float step = lr * g;
        theta[j] = theta[j] - step;
    }
    return ORC_OK;
}

uint32_t orc_sizeof_params(void) { return (uint32_t)sizeof(orc_params_t); }
uint32_t orc_sizeof_stats(void) { return (uint32_t)sizeof(orc_stats_t); }
