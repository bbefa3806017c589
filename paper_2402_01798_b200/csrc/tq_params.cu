// Parameter design: statistics -> truncation threshold alpha and codebook, on the host (tq_params,
// tq_params_batch, tq_params_from_levels) and, with the same code, on the device (tq_params_device:
// one thread per worker, so a round needs no host round trip between statistics and compression).
//
// Follows Section 4 of the paper.  The gradient density is modelled as a power-law tail
// p(g) = rho (gamma-1) g_min^(gamma-1) |g|^-gamma beyond g_min (Section 4.1, tail model), with rho
// the one-sided tail mass, completed by a flat body p = (1 - 2 rho) / (2 g_min) below g_min so that
// Q_U, Q_N and the p^(1/3) density of Section 4.2 are defined on the whole of [-alpha, alpha].
// Everything here is O(L) double-precision work per worker; results are rounded once to fp32.
// Host and device use their own pow / log / exp / cbrt, so the two can differ in the last fp32 bit
// of alpha or of a level; each is a valid quantizer, and a packed buffer is always decoded with the
// parameters it was encoded with.
#include <cmath>

#include "tq.h"
#include "tq_launch.h"

namespace tq {

#define TQ_HD __host__ __device__

struct TailModel {
    double g_min, rho, gamma;
    // constants of the model, formed once (the alpha iteration evaluates q_of() many times):
    double cb;       // body height^(1/3):       ((1 - 2 rho) / (2 g_min))^(1/3)
    double coef;     // p^(1/3) = coef * |g|^(-gamma/3) in the tail
    double b;        // 1 - gamma/3
    double gmin_b;   // g_min^b

    TQ_HD TailModel(double g_min_, double rho_, double gamma_) : g_min(g_min_), rho(rho_), gamma(gamma_) {
        cb = cbrt((1.0 - 2.0 * rho) / (2.0 * g_min));
        coef = cbrt(rho * (gamma - 1.0)) * pow(g_min, (gamma - 1.0) / 3.0);
        b = 1.0 - gamma / 3.0;
        gmin_b = pow(g_min, b);
    }

    // mass inside [-a, a]  (Q_U of Section 4.1)
    TQ_HD double mass_inside(double a) const {
        if (a <= g_min) return (1.0 - 2.0 * rho) * (a / g_min);
        return 1.0 - 2.0 * rho * pow(a / g_min, 1.0 - gamma);
    }
    // integral of p^(1/3) over [0, x]
    TQ_HD double cuberoot_integral(double x) const {
        if (x <= g_min) return cb * x;
        const double tail = (b == 0.0) ? coef * log(x / g_min) : coef * (pow(x, b) - gmin_b) / b;
        return cb * g_min + tail;
    }
    // x with cuberoot_integral(x) = tau, tau >= 0
    TQ_HD double cuberoot_integral_inverse(double tau) const {
        const double at_gmin = cb * g_min;
        if (tau <= at_gmin) return tau / cb;
        const double rest = (tau - at_gmin) / coef;
        if (b == 0.0) return g_min * exp(rest);
        return pow(gmin_b + b * rest, 1.0 / b);
    }
    // Q_N of Section 4.2: [ int_{-a}^{a} p^(1/3) (1/(2a))^(2/3) ]^3 = (2 I)^3 / (2a)^2
    TQ_HD double holder_factor(double a) const {
        const double two_i = 2.0 * cuberoot_integral(a);
        return two_i * two_i * two_i / (4.0 * a * a);
    }
    // Q_B of the Appendix for the split at k * a: inner and outer mass, each spread evenly
    TQ_HD double biscaled_factor(double a, double k) const {
        const double inner = mass_inside(k * a);
        double outer = mass_inside(a) - inner;
        if (outer < 0.0) outer = 0.0;
        const double t = cbrt(outer) * pow(1.0 - k, 2.0 / 3.0) + cbrt(inner) * pow(k, 2.0 / 3.0);
        return t * t * t;
    }
    // d/dx of mass_inside: twice the model density
    TQ_HD double mass_slope(double x) const {
        if (x <= g_min) return (1.0 - 2.0 * rho) / g_min;
        return 2.0 * rho * (gamma - 1.0) / g_min * pow(x / g_min, -gamma);
    }
    // A quantity with the sign of dQ_B/dk on 0 < k < 1.  With u = mass_inside(k a), w = mass_inside(a) - u and
    // Q_B^(1/3) = w^(1/3) (1-k)^(2/3) + u^(1/3) k^(2/3), the derivative times the positive factor
    // 3 w^(2/3) (1-k)^(1/3) u^(2/3) k^(1/3) is
    //     w^(2/3) (1-k)^(1/3) (u' k + 2 u)  -  u^(2/3) k^(1/3) (u' (1-k) + 2 w),      u' = a * mass_slope(k a).
    TQ_HD double biscaled_slope_sign(double a, double k) const {
        const double u = mass_inside(k * a);
        double w = mass_inside(a) - u;
        if (w < 0.0) w = 0.0;
        const double du = a * mass_slope(k * a);
        const double cw = cbrt(w), cu = cbrt(u);
        return cw * cw * cbrt(1.0 - k) * (du * k + 2.0 * u) - cu * cu * cbrt(k) * (du * (1.0 - k) + 2.0 * w);
    }
    // k* = argmin_k Q_B(a, k) (Appendix).  Q_B(a, 0) = Q_B(a, 1) = Q_U(a), so the minimum is a point where the
    // slope turns from negative to positive (at the density's jump, k a = g_min, it may do so without
    // passing through zero).  Every such turn between neighbours of a 128-point grid is closed in on by
    // bisection of the slope's sign; the turn with the smallest Q_B wins.  No turn: the minimum is an end.
    TQ_HD double biscaled_split(double a) const {
        constexpr int kGrid = 128;
        double best_k = 0.0, best_q = biscaled_factor(a, 0.0);
        constexpr double kFirst = 9.094947017729282e-13;                // 2^-40: the grid's first point, in place of 0
        bool prev_neg = biscaled_slope_sign(a, kFirst) < 0.0;        // slope at the previous grid point was negative
        for (int j = 1; j <= kGrid; ++j) {
            const double k = static_cast<double>(j) / kGrid;
            // at k = 1 the slope's sign is that of approaching the end from inside: treat the end as a turn
            const bool neg = j < kGrid ? biscaled_slope_sign(a, k) < 0.0 : false;
            if (prev_neg && !neg) {
                double lo = j > 1 ? static_cast<double>(j - 1) / kGrid : kFirst, hi = k;      // slope < 0 at lo, >= 0 at hi
                for (int it = 0; it < 64 && hi - lo > 0.0; ++it) {
                    const double mid = 0.5 * (lo + hi);
                    if (mid <= lo || mid >= hi) break;
                    if (biscaled_slope_sign(a, mid) < 0.0) lo = mid; else hi = mid;
                }
                const double kk = 0.5 * (lo + hi), q = biscaled_factor(a, kk);
                if (q < best_q) { best_q = q; best_k = kk; }
            }
            prev_neg = neg;
        }
        return best_k;
    }
    TQ_HD double q_of(uint32_t mode, double a) const {
        if (mode == TQ_UNIFORM) return mass_inside(a);
        if (mode == TQ_NONUNIFORM) return holder_factor(a);
        return biscaled_factor(a, biscaled_split(a));
    }
    // right-hand side of the boxed alpha equations for a given Q
    TQ_HD double alpha_for_q(double s, double q) const {
        return g_min * pow(2.0 * rho * s * s / ((gamma - 2.0) * q), 1.0 / (gamma - 1.0));
    }
};

TQ_HD inline bool finite_f(float x) { return fabsf(x) <= 3.402823466e38f; }
TQ_HD inline bool finite_d(double x) { return fabs(x) <= 1.7976931348623157e308; }

TQ_HD inline float ceil_to_float(double v) {
    float f = static_cast<float>(v);
    if (static_cast<double>(f) < v) f = nextafterf(f, 3.402823466e38f * 2.0f);   // towards +inf
    return f;
}

// inv_width / inv_step from a finished level table.  Rounded up so that a value sitting on the
// top level maps to probability >= 1 and is reproduced exactly.
TQ_HD inline tq_status finish(tq_params_t* p) {
    const uint32_t s = p->num_levels - 1;
    for (uint32_t k = 0; k < s; ++k) {
        if (!(p->levels[k + 1] > p->levels[k])) return TQ_ERR_DEGENERATE_LEVELS;
        const float w = static_cast<float>(static_cast<double>(p->levels[k + 1]) - static_cast<double>(p->levels[k]));
        p->inv_width[k] = ceil_to_float(1.0 / static_cast<double>(w));
        if (!finite_f(p->inv_width[k])) return TQ_ERR_DEGENERATE_LEVELS;
    }
    p->alpha = p->levels[s];
    p->inv_step = ceil_to_float(static_cast<double>(s) / static_cast<double>(2.0f * p->alpha));
    if (!finite_f(p->inv_step)) return TQ_ERR_DEGENERATE_LEVELS;
    return TQ_OK;
}

TQ_HD inline bool bits_for_levels(uint32_t num_levels, uint32_t* bits) {
    for (uint32_t b = 1; b <= 4; ++b)
        if ((1u << b) == num_levels) { *bits = b; return true; }
    return false;
}

TQ_HD inline void clear(tq_params_t* p) {
    p->bits = p->num_levels = p->mode = p->flags = 0;
    p->alpha = p->inv_step = p->gamma = p->g_min = p->rho = 0.0f;
    p->iterations = 0; p->reserved[0] = p->reserved[1] = 0.0f;
    for (int k = 0; k < TQ_MAX_LEVELS; ++k) { p->levels[k] = 0.0f; p->inv_width[k] = 0.0f; }
}

// Section 4 as a whole for one worker.  Arguments are already range-checked.
TQ_HD inline tq_status design(const tq_stats_t* st, uint32_t num_levels, uint32_t bits, uint32_t mode, double gamma,
                              int rule, double alpha_user, tq_params_t* out) {
    clear(out);
    out->bits = bits; out->num_levels = num_levels; out->mode = mode;
    const double s = static_cast<double>(num_levels - 1);

    if (gamma != gamma) {  // NaN: Section 5, gamma = 1 + n / sum ln(g_j / g_min)
        if (st->n_tail == 0 || !(st->sum_log_tail > 0.0)) return TQ_ERR_DOMAIN;
        gamma = 1.0 + static_cast<double>(st->n_tail) / st->sum_log_tail;
        out->flags |= TQ_FLAG_GAMMA_FROM_MLE;
    }
    if (!(gamma > 2.0) || !finite_d(gamma)) return TQ_ERR_DOMAIN;
    if (!(st->g_min > 0.0f) || !finite_f(st->g_min) || st->d == 0) return TQ_ERR_DOMAIN;
    const double rho = static_cast<double>(st->n_tail) / (2.0 * static_cast<double>(st->d));
    if (!(rho > 0.0) || !(rho < 0.5)) return TQ_ERR_DOMAIN;
    const TailModel m(static_cast<double>(st->g_min), rho, gamma);
    out->gamma = static_cast<float>(gamma); out->g_min = st->g_min; out->rho = static_cast<float>(rho);

    double alpha;
    if (rule == TQ_ALPHA_USER) {
        if (!(alpha_user > 0.0) || !finite_d(alpha_user)) return TQ_ERR_DOMAIN;
        alpha = alpha_user;
    } else if (rule == TQ_ALPHA_MAXABS) {                    // Section 5 baselines: no truncation
        if (!(st->max_abs > 0.0f)) return TQ_ERR_DOMAIN;
        alpha = static_cast<double>(st->max_abs);
    } else {
        const double cap = static_cast<double>(st->max_abs);
        alpha = m.alpha_for_q(s, 1.0);                       // alpha'
        if (rule == TQ_ALPHA_FIXED_POINT) {
            // Iterate alpha <- F(alpha) (the boxed equation with Q evaluated at the current alpha) until a
            // plain step changes alpha by <= 1e-12 relative.  The plain iteration converges linearly (70+
            // steps for gamma = 3, s = 15), so every pair of steps is followed by Aitken's extrapolation
            // to the limit of the geometric sequence when the steps are monotone and contracting; the
            // result is still accepted only through the plain-step test, so it is the same fixed point.
            int it = 0;
            while (it < 10000) {
                if (cap > 0.0 && alpha > cap) break;         // no fixed point below max|g|
                const double a1 = m.alpha_for_q(s, m.q_of(mode, alpha));
                ++it;
                const double d1 = a1 - alpha;
                alpha = a1;
                if (fabs(d1) <= 1e-12 * fabs(a1)) break;
                if (cap > 0.0 && alpha > cap) break;
                const double a2 = m.alpha_for_q(s, m.q_of(mode, a1));
                ++it;
                const double d2 = a2 - a1;
                alpha = a2;
                if (fabs(d2) <= 1e-12 * fabs(a2)) break;
                const double r = d2 / d1;
                if (r > 0.0 && r < 0.999) {
                    const double limit = a2 + d2 * r / (1.0 - r);
                    if (limit > 0.0 && finite_d(limit) && !(cap > 0.0 && limit > cap)) alpha = limit;
                }
            }
            out->iterations = it;
        }
        if (alpha != alpha) return TQ_ERR_DOMAIN;
        if (alpha < m.g_min) { alpha = m.g_min; out->flags |= TQ_FLAG_ALPHA_AT_GMIN; }
        if (cap > 0.0 && alpha > cap) { alpha = cap; out->flags |= TQ_FLAG_ALPHA_CAPPED; }
    }

    const float alpha_f = static_cast<float>(alpha);
    if (!(alpha_f > 0.0f) || !finite_f(2.0f * alpha_f)) return TQ_ERR_DOMAIN;
    const double a = static_cast<double>(alpha_f);
    const uint32_t si = num_levels - 1;
    if (mode == TQ_UNIFORM) {
        const double step = 2.0 * a / s;                     // Section 4.1 codebook
        for (uint32_t k = 0; k <= si; ++k) out->levels[k] = static_cast<float>(-a + static_cast<double>(k) * step);
    } else if (mode == TQ_BISCALED) {
        // Appendix: density s c_in / D inside k* alpha and s c_out / D outside, c = (mean density)^(1/3),
        // D = 2 alpha (c_out (1 - k*) + c_in k*).  Level k sits where the density accumulated from the
        // centre reaches k - s/2.  Upper half, then mirrored.
        const double k = m.biscaled_split(a), beta = k * a;
        const double c_in = cbrt(m.mass_inside(beta) / (2.0 * beta));
        const double c_out = cbrt((m.mass_inside(a) - m.mass_inside(beta)) / (2.0 * (a - beta)));
        const double denom = 2.0 * a * (c_out * (1.0 - k) + c_in * k);
        const double lam_in = s * c_in / denom, lam_out = s * c_out / denom;
        for (uint32_t j = (si + 1) / 2; j <= si; ++j) {
            const double c = static_cast<double>(j) - 0.5 * s;
            const double x = c <= lam_in * beta ? c / lam_in : beta + (c - lam_in * beta) / lam_out;
            out->levels[j] = static_cast<float>(x);
            out->levels[si - j] = -static_cast<float>(x);
        }
    } else {
        // lambda_s = s p^(1/3) / int p^(1/3): level k sits where the running integral of p^(1/3)
        // from the centre reaches (2k/s - 1) of its value at alpha.  Upper half, then mirrored.
        const double total = m.cuberoot_integral(a);
        for (uint32_t k = (si + 1) / 2; k <= si; ++k) {
            const double tau = (2.0 * static_cast<double>(k) / s - 1.0) * total;
            const float l = static_cast<float>(m.cuberoot_integral_inverse(tau));
            out->levels[k] = l;
            out->levels[si - k] = -l;
        }
    }
    out->levels[0] = -alpha_f;
    out->levels[si] = alpha_f;
    return finish(out);
}

static bool valid_request(uint32_t num_levels, int mode, int rule, uint32_t* bits) {
    if (!bits_for_levels(num_levels, bits)) return false;
    if (mode != TQ_UNIFORM && mode != TQ_NONUNIFORM && mode != TQ_BISCALED) return false;
    return rule == TQ_ALPHA_CLOSED || rule == TQ_ALPHA_FIXED_POINT || rule == TQ_ALPHA_USER || rule == TQ_ALPHA_MAXABS;
}

// One thread per worker.  A worker whose statistics are outside the model's domain gets
// flags = TQ_FLAG_INVALID, iterations = the status code, alpha = 0 and an all-zero codebook.
__global__ void params_kernel(const tq_stats_t* __restrict__ stats, uint32_t n, uint32_t num_levels, uint32_t bits,
                              uint32_t mode, double gamma, int rule, double alpha_user, tq_params_t* __restrict__ out) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const tq_stats_t st = stats[i];
    tq_params_t p;
    const tq_status s = design(&st, num_levels, bits, mode, gamma, rule, alpha_user, &p);
    if (s != TQ_OK) {
        clear(&p);
        p.bits = bits; p.num_levels = num_levels; p.mode = mode;
        p.flags = TQ_FLAG_INVALID; p.iterations = static_cast<int32_t>(s);
    }
    out[i] = p;
}

cudaError_t launch_params_device(const tq_stats_t* stats_dev, uint32_t n, uint32_t num_levels, uint32_t bits, uint32_t mode,
                                 double gamma, int rule, double alpha_user, tq_params_t* params_dev, cudaStream_t stream) {
    params_kernel<<<(n + 31) / 32, 32, 0, stream>>>(stats_dev, n, num_levels, bits, mode, gamma, rule, alpha_user, params_dev);
    return cudaGetLastError();
}

bool params_request_ok(uint32_t num_levels, int mode, int rule, uint32_t* bits) { return valid_request(num_levels, mode, rule, bits); }

}  // namespace tq

extern "C" tq_status tq_params_from_levels(const float* levels_host, uint32_t num_levels, tq_mode mode,
                                           tq_params_t* out) {
    uint32_t bits = 0;
    if (!levels_host || !out || !tq::bits_for_levels(num_levels, &bits)) return TQ_ERR_INVALID_ARG;
    if (mode != TQ_UNIFORM && mode != TQ_NONUNIFORM && mode != TQ_BISCALED) return TQ_ERR_INVALID_ARG;
    tq::clear(out);
    out->bits = bits; out->num_levels = num_levels; out->mode = mode;
    for (uint32_t k = 0; k < num_levels; ++k) out->levels[k] = levels_host[k];
    const float top = levels_host[num_levels - 1];
    if (!(top > 0.0f) || !tq::finite_f(2.0f * top) || levels_host[0] != -top) return TQ_ERR_DOMAIN;
    return tq::finish(out);
}

extern "C" tq_status tq_params(const tq_stats_t* st, uint32_t num_levels, tq_mode mode, double gamma,
                               tq_alpha_rule rule, double alpha_user, tq_params_t* out) {
    uint32_t bits = 0;
    if (!st || !out || !tq::valid_request(num_levels, mode, rule, &bits)) return TQ_ERR_INVALID_ARG;
    return tq::design(st, num_levels, bits, mode, gamma, rule, alpha_user, out);
}

extern "C" tq_status tq_params_batch(const tq_stats_t* st, uint32_t n_workers, uint32_t num_levels, tq_mode mode,
                                     double gamma, tq_alpha_rule rule, double alpha_user, tq_params_t* out) {
    if (!st || !out || n_workers == 0 || n_workers > TQ_MAX_WORKERS) return TQ_ERR_INVALID_ARG;
    for (uint32_t i = 0; i < n_workers; ++i)
        if (tq_status s = tq_params(st + i, num_levels, mode, gamma, rule, alpha_user, out + i)) return s;
    return TQ_OK;
}
