"""Pins for the oracle's parameter design (Section 4: alpha and the quantization density).

The oracle evaluates closed forms.  They are pinned here by routes that do not use those
closed forms: numerical quadrature of the defining integrals (Lemma 2's error term, the
definitions of Q_U, Q_N and rho), brute-force minimisation over alpha and over perturbed
densities, the worked numbers obtained by hand below, and sampling from exact Pareto tails.
"""
import math

import numpy as np
import pytest
from scipy import integrate, optimize

F32 = np.float32

MODELS = [  # (g_min, rho, gamma)
    (1.0, 0.10, 4.0),
    (1e-3, 0.06, 3.5),
    (2e-4, 0.15, 5.0),
    (1e-3, 0.12, 3.2),
]
LOW_GAMMA = [(1e-3, 0.10, 3.0), (1e-3, 0.14, 2.5), (5e-4, 0.08, 2.2)]


def _quad(f, a, b, **kw):
    return integrate.quad(f, a, b, limit=400, epsabs=0, epsrel=1e-11, **kw)[0]


def _pdf(orc, m):
    return lambda g: orc.model_fn("model_pdf", m, g)


# ------------------------------------------------------------------ the density model
@pytest.mark.parametrize("gm,rho,gamma", MODELS + LOW_GAMMA)
def test_density_is_normalised_and_rho_is_one_sided_tail_mass(orc, gm, rho, gamma):
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    body = 2 * _quad(pdf, 0, gm)
    tail = _quad(pdf, gm, gm * 1e3) + _quad(pdf, gm * 1e3, np.inf)
    assert abs(tail - rho) < 1e-8          # rho = integral_{g_min}^inf p (text under the tail model)
    assert abs(body + 2 * tail - 1.0) < 1e-8
    # tail follows rho * f(x | gamma, g_min) with f the power-law density of Definition 1
    x = 3.7 * gm
    assert math.isclose(pdf(x), rho * (gamma - 1) / gm ** (1 - gamma) * x ** (-gamma), rel_tol=1e-12)
    assert pdf(-x) == pdf(x)


@pytest.mark.parametrize("gm,rho,gamma", MODELS + LOW_GAMMA)
def test_QU_QN_H_are_their_defining_integrals(orc, gm, rho, gamma):
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    for alpha in (0.4 * gm, gm, 1.7 * gm, 9.0 * gm, 60.0 * gm):
        pts = [gm] if alpha > gm else None
        qu = 2 * _quad(pdf, 0, alpha, points=pts)
        assert math.isclose(orc.model_fn("model_QU", m, alpha), qu, rel_tol=1e-9)
        h = _quad(lambda g: pdf(g) ** (1 / 3), 0, alpha, points=pts)
        assert math.isclose(orc.model_fn("model_H", m, alpha), h, rel_tol=1e-9)
        assert math.isclose(orc.model_fn("model_Hinv", m, h), alpha, rel_tol=1e-8)
        qn = (2 * _quad(lambda g: pdf(g) ** (1 / 3) * (1 / (2 * alpha)) ** (2 / 3), 0, alpha, points=pts)) ** 3
        assert math.isclose(orc.model_fn("model_QN", m, alpha), qn, rel_tol=1e-8)
        assert qn <= qu * (1 + 1e-9) <= 1 + 1e-9          # Hoelder step after Theorem 2


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
def test_truncation_bias_and_uniform_error_are_lemma2_integrals(orc, gm, rho, gamma):
    """E_TQ N/d = (1/4) int_{-a}^{a} p / lambda^2 + 2 int_a^inf (g-a)^2 p   (Lemma 2),
    with lambda = s / (2a): must equal the Section 4.1 error equation."""
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    for s in (3, 7, 15):
        for alpha in (1.2 * gm, 2.5 * gm, 11.0 * gm):
            bias = 2 * (_quad(lambda g: (g - alpha) ** 2 * pdf(g), alpha, alpha * 1e3)
                        + _quad(lambda g: (g - alpha) ** 2 * pdf(g), alpha * 1e3, np.inf))
            assert math.isclose(orc.model_fn("truncation_bias", m, alpha), bias, rel_tol=1e-6)
            lam = s / (2 * alpha)
            var = 0.25 * 2 * _quad(lambda g: pdf(g) / lam ** 2, 0, alpha, points=[gm])
            assert math.isclose(orc.model_fn("etq_uniform", m, alpha, s), var + bias, rel_tol=1e-6)


# ------------------------------------------------------------------ uniform alpha
def test_worked_example_uniform(orc):
    """gamma = 4, g_min = 1, rho = 0.1, s = 7, by hand:
    C = 2 rho s^2 / (gamma-2) = 4.9, alpha' = 4.9^(1/3);
    the boxed equation with Q_U = 1 - 2 rho (alpha/g_min)^(1-gamma) reads y = C / (1 - 2 rho / y)
    for y = alpha^3, i.e. y = C + 2 rho = 5.1; Q_U = 1 - 0.2/5.1;
    error equation: Q_U alpha^2 / 49 + 4 rho / (2 * 1) / alpha."""
    m = orc.Model(1.0, 0.1, 4.0)
    assert math.isclose(orc.alpha_prime(m, 7), 4.9 ** (1 / 3), rel_tol=1e-14)
    a, iters, capped = orc.alpha_fixed_point(m, 7, orc.UNIFORM)
    assert math.isclose(a, 5.1 ** (1 / 3), rel_tol=1e-11) and not capped and iters < 50
    qu = 1 - 0.2 / 5.1
    assert math.isclose(orc.model_fn("model_QU", m, a), qu, rel_tol=1e-11)
    e = qu * 5.1 ** (2 / 3) / 49 + 0.2 / 5.1 ** (1 / 3)
    assert math.isclose(orc.model_fn("etq_uniform", m, a, 7), e, rel_tol=1e-11)
    assert math.isclose(orc.model_fn("etq_theorem", m, qu, 7), e, rel_tol=1e-11)   # Theorem 1
    assert abs(e - 0.174287) < 1e-6


@pytest.mark.parametrize("gm,rho,gamma", MODELS + LOW_GAMMA)
@pytest.mark.parametrize("s", [3, 7, 15])
def test_uniform_fixed_point_solves_boxed_equation(orc, gm, rho, gamma, s):
    m = orc.Model(gm, rho, gamma)
    a, iters, capped = orc.alpha_fixed_point(m, s, orc.UNIFORM)
    y = 2 * rho * (s * s + gamma - 2) / (gamma - 2)         # closed form of the fixed point, valid when y > 1
    if y > 1:
        assert math.isclose(a, gm * y ** (1 / (gamma - 1)), rel_tol=1e-10)
    qu = 2 * _quad(_pdf(orc, m), 0, a, points=[gm] if a > gm else None)
    rhs = gm * (2 * rho * s * s / ((gamma - 2) * qu)) ** (1 / (gamma - 1))
    assert math.isclose(a, rhs, rel_tol=1e-8)
    assert a >= orc.alpha_prime(m, s) * (1 - 1e-12)          # Q_U <= 1 can only raise alpha


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
@pytest.mark.parametrize("s", [3, 7, 15])
def test_boxed_alpha_minimises_error_with_Q_frozen(orc, gm, rho, gamma, s):
    """Proof of Theorem 1: minimising Q alpha^2/s^2 + bias(alpha) over alpha (Q held at its value
    at the optimum) gives the boxed alpha, and the minimum is Theorem 1's expression.
    Brute force: bounded scalar minimisation of the quadrature-built objective."""
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    a_star, _, _ = orc.alpha_fixed_point(m, s, orc.UNIFORM)
    if a_star <= gm:
        pytest.skip("optimum inside the body: the tail formulas do not apply")
    q = orc.model_fn("model_QU", m, a_star)

    def objective(alpha):
        bias = 2 * (_quad(lambda g: (g - alpha) ** 2 * pdf(g), alpha, alpha * 1e3)
                    + _quad(lambda g: (g - alpha) ** 2 * pdf(g), alpha * 1e3, np.inf))
        return q * alpha ** 2 / s ** 2 + bias

    res = optimize.minimize_scalar(objective, bounds=(gm, 50 * a_star), method="bounded",
                                   options={"xatol": 1e-10 * a_star})
    assert math.isclose(res.x, a_star, rel_tol=2e-5)
    assert math.isclose(res.fun, orc.model_fn("etq_theorem", m, q, s), rel_tol=1e-7)
    assert math.isclose(orc.model_fn("etq_uniform", m, a_star, s), orc.model_fn("etq_theorem", m, q, s), rel_tol=1e-9)


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
def test_alpha_prime_error_coefficient_and_epsilon_bound(orc, gm, rho, gamma):
    """Text after Theorem 1: with alpha' the error is [(gamma-3) Q_U(alpha') + 2] * K, against
    (gamma-1) Q_U(alpha)^((gamma-3)/(gamma-1)) * K at the optimum; the gap is <= 2 [1 - Q_U(alpha')] K."""
    s = 7
    m = orc.Model(gm, rho, gamma)
    ap = orc.alpha_prime(m, s)
    a, _, _ = orc.alpha_fixed_point(m, s, orc.UNIFORM)
    if ap <= gm:
        pytest.skip("alpha' inside the body")
    K = gm ** 2 * (2 * rho) ** (2 / (gamma - 1)) * s ** ((6 - 2 * gamma) / (gamma - 1)) \
        / ((gamma - 3) * (gamma - 2) ** (2 / (gamma - 1)))
    qp, qa = orc.model_fn("model_QU", m, ap), orc.model_fn("model_QU", m, a)
    assert math.isclose(orc.model_fn("etq_uniform", m, ap, s), ((gamma - 3) * qp + 2) * K, rel_tol=1e-9)
    eps = (gamma - 3) * qp + 2 - (gamma - 1) * qa ** ((gamma - 3) / (gamma - 1))
    # the paper bounds the gap from above only (alpha solves the equation with Q frozen, so the
    # varying-Q error at alpha' can be marginally smaller)
    assert eps <= 2 * (1 - qp) + 1e-12 and abs(eps) <= 2 * (1 - qp) + 1e-12


# ------------------------------------------------------------------ non-uniform density, alpha, levels
@pytest.mark.parametrize("gm,rho,gamma", MODELS + LOW_GAMMA[:1])
def test_cube_root_density_minimises_quantization_variance(orc, gm, rho, gamma):
    """Boxed density: among densities with integral s over [-alpha, alpha], lambda ~ p^(1/3)
    minimises int p / lambda^2.  Brute force: its value is Q_N (2 alpha)^2 / s^2 * ... and any
    admissible perturbation (uniform; blends; p^(1/2); p^(1/4)) is worse."""
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    alpha, s = 12.0 * gm, 15

    def variance_for(shape):
        norm = 2 * _quad(shape, 0, alpha, points=[gm])
        return 0.25 * 2 * _quad(lambda g: pdf(g) / (s * shape(g) / norm) ** 2, 0, alpha, points=[gm])

    best = variance_for(lambda g: pdf(g) ** (1 / 3))
    assert math.isclose(best, orc.model_fn("model_QN", m, alpha) * alpha ** 2 / s ** 2, rel_tol=1e-7)
    bias = orc.model_fn("truncation_bias", m, alpha) if gamma > 3 else 0.0
    if gamma > 3:
        assert math.isclose(orc.model_fn("etq_nonuniform", m, alpha, s), best + bias, rel_tol=1e-7)
    for other in (lambda g: 1.0, lambda g: pdf(g) ** 0.5, lambda g: pdf(g) ** 0.25,
                  lambda g: 0.5 * pdf(g) ** (1 / 3) + 0.5 * pdf(alpha) ** (1 / 3),
                  lambda g: pdf(g) ** (1 / 3) * (1 + 0.2 * math.sin(5 * g / alpha))):
        assert variance_for(other) > best * (1 + 1e-6)


@pytest.mark.parametrize("gm,rho,gamma", MODELS + LOW_GAMMA)
@pytest.mark.parametrize("L", [4, 8, 16])
def test_levels_split_the_density_into_equal_shares(orc, gm, rho, gamma, L):
    """integral of lambda_s over each cell is 1 (density <-> codebook, Section 3.1), i.e. the
    integral of p^(1/3) between consecutive levels is 2 H(alpha) / s; levels are antisymmetric,
    end at +-alpha, and zero is not a level (s odd)."""
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    s = L - 1
    for alpha in (1.5 * gm, 8.0 * gm, 40.0 * gm):
        p = orc.build_table(m, L, orc.NONUNIFORM, alpha)
        lv = p.levels_np().astype(np.float64)
        assert lv[0] == -p.alpha and lv[-1] == p.alpha and np.all(np.diff(lv) > 0)
        assert np.array_equal(lv, -lv[::-1])
        assert not np.any(lv == 0.0)
        share = 2 * _quad(lambda g: pdf(g) ** (1 / 3), 0, p.alpha, points=[gm]) / s
        for k in range(s):
            a, b = lv[k], lv[k + 1]
            pts = [x for x in (-gm, gm) if a < x < b] or None
            cell = _quad(lambda g: pdf(g) ** (1 / 3), a, b, points=pts)
            assert math.isclose(cell, share, rel_tol=2e-6), (alpha, k)


@pytest.mark.parametrize("L", [4, 8, 16])
def test_flat_density_gives_uniform_levels(orc, L):
    """Special case: for alpha <= g_min the model density is flat on [-alpha, alpha], the boxed
    density is the constant s / (2 alpha), and the codebook is the uniform one of Section 4.1."""
    m = orc.Model(1e-3, 0.1, 3.5)
    pn = orc.build_table(m, L, orc.NONUNIFORM, 8e-4)
    pu = orc.build_table(m, L, orc.UNIFORM, 8e-4)
    assert np.allclose(pn.levels_np(), pu.levels_np(), rtol=3e-7, atol=0)
    s = L - 1
    want = -8e-4 + np.arange(L) * 2 * 8e-4 / s
    assert np.allclose(pu.levels_np(), want.astype(F32), rtol=2e-7, atol=1e-12)
    assert math.isclose(pu.inv_step, s / (2 * float(F32(8e-4))), rel_tol=2e-7)
    assert pu.inv_step >= s / (2 * float(F32(8e-4)))          # rounded up (R11)


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
@pytest.mark.parametrize("s", [3, 7, 15])
def test_nonuniform_fixed_point_and_theorem2(orc, gm, rho, gamma, s):
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    a, iters, capped = orc.alpha_fixed_point(m, s, orc.NONUNIFORM)
    assert not capped and iters < 10000
    qn = (2 * _quad(lambda g: pdf(g) ** (1 / 3) * (1 / (2 * a)) ** (2 / 3), 0, a, points=[gm] if a > gm else None)) ** 3
    rhs = gm * (2 * rho * s * s / ((gamma - 2) * qn)) ** (1 / (gamma - 1))
    assert math.isclose(a, rhs, rel_tol=1e-7)
    au, _, _ = orc.alpha_fixed_point(m, s, orc.UNIFORM)
    assert a >= au * (1 - 1e-9)                               # "TNQSGD uses a larger truncation threshold"
    if a > gm:
        e_n = orc.model_fn("etq_nonuniform", m, a, s)
        assert math.isclose(e_n, orc.model_fn("etq_theorem", m, qn, s), rel_tol=1e-6)   # Theorem 2
        assert e_n <= orc.model_fn("etq_uniform", m, au, s) * (1 + 1e-9)                # lower error than uniform


@pytest.mark.parametrize("gm,rho,gamma", MODELS + LOW_GAMMA[:1])
def test_nonuniform_table_has_lower_model_distortion_than_uniform(orc, gm, rho, gamma):
    """Exact per-element variance (x - l_{k-1})(l_k - x) (proof of Lemma 1) integrated against the
    model density: the p^(1/3) codebook beats the uniform one at the same alpha and s."""
    m = orc.Model(gm, rho, gamma)
    pdf = _pdf(orc, m)
    alpha = 15 * gm

    def distortion(p):
        lv = p.levels_np().astype(np.float64)
        tot = 0.0
        for k in range(len(lv) - 1):
            a, b = lv[k], lv[k + 1]
            pts = [x for x in (-gm, gm) if a < x < b] or None
            tot += _quad(lambda x: (x - a) * (b - x) * pdf(x), a, b, points=pts)
        return tot

    for L in (8, 16):
        dn = distortion(orc.build_table(m, L, orc.NONUNIFORM, alpha))
        du = distortion(orc.build_table(m, L, orc.UNIFORM, alpha))
        assert dn < du


def test_slow_convergence_and_divergence_are_capped(orc):
    """For gamma < 3 the non-uniform map grows linearly in alpha with slope
    [s^2 beta^3 / ((gamma-2)(gamma-1))]^(1/(gamma-1)) asymptotically (beta = 1 - gamma/3); when that
    exceeds 1 there is no finite fixed point and the iteration must stop at the cap."""
    m = orc.Model(1e-3, 0.1, 2.2)
    beta = 1 - 2.2 / 3
    slope = (15 ** 2 * beta ** 3 / (0.2 * 1.2)) ** (1 / 1.2)
    assert slope > 1
    a, iters, capped = orc.alpha_fixed_point(m, 15, orc.NONUNIFORM, cap=5.0)
    assert capped and a > 5.0 and iters < 10000
    st = orc.Stats(d=1000, n_tail=200, n_nonfinite=0, sum_abs=1.0, sum_sq=1.0, sum_log_tail=200 / 1.2,
                   max_abs=5.0, g_min=1e-3)
    p = orc.params(st, 16, orc.NONUNIFORM, gamma=2.2)
    assert p.flags & orc.FLAG_ALPHA_CAPPED and p.alpha == 5.0
    # and a convergent low-gamma case still satisfies its equation
    m2 = orc.Model(1e-3, 0.1, 2.5)
    a2, it2, cap2 = orc.alpha_fixed_point(m2, 7, orc.NONUNIFORM)
    assert not cap2
    assert math.isclose(a2, 1e-3 * (2 * 0.1 * 49 / (0.5 * orc.model_fn("model_QN", m2, a2))) ** (1 / 1.5), rel_tol=1e-9)


# ------------------------------------------------------------------ statistics -> parameters
def _pareto_symmetric(rng, d, gm, rho, gamma):
    """Samples from the model density itself: flat body, exact Pareto tails (inverse-CDF)."""
    u = rng.random(d)
    tail = u < 2 * rho
    mag = np.where(tail, gm * (1 - rng.random(d)) ** (-1 / (gamma - 1)), gm * rng.random(d))
    return (mag * np.where(rng.random(d) < 0.5, -1, 1)).astype(F32)


@pytest.mark.parametrize("gamma", [2.5, 3.0, 4.0])
def test_hill_estimator_and_rho_on_exact_pareto_tails(orc, gamma):
    """gamma_hat = 1 + n / sum ln(g_j / g_min) (Section 5) recovers gamma; rho_hat = n / (2d)."""
    rng = np.random.default_rng(int(gamma * 10))
    d, gm, rho = 400_000, 1e-3, 0.11
    g = _pareto_symmetric(rng, d, gm, rho, gamma)
    st = orc.stats(g, g_min=gm)
    n = st.n_tail
    assert abs(n / (2 * d) - rho) < 4 * math.sqrt(2 * rho / d)
    p = orc.params(st, 8, orc.UNIFORM)                       # gamma = NaN -> MLE
    assert p.flags & orc.FLAG_GAMMA_FROM_MLE
    assert abs(p.gamma - gamma) < 4 * (gamma - 1) / math.sqrt(n)
    assert math.isclose(p.rho, n / (2 * d), rel_tol=1e-6)


def test_stats_match_numpy(orc):
    rng = np.random.default_rng(11)
    g = (rng.standard_t(3.0, 100_003) * 1e-3).astype(F32)
    g[[5, 77, 1000]] = [np.nan, np.inf, -np.inf]
    st = orc.stats(g)                                        # automatic g_min = mean |g|
    fin = g[np.isfinite(g)].astype(np.float64)
    assert st.d == g.size and st.n_nonfinite == 3
    assert math.isclose(st.sum_abs, np.abs(fin).sum(), rel_tol=1e-12)
    assert math.isclose(st.sum_sq, (fin ** 2).sum(), rel_tol=1e-12)
    assert st.max_abs == float(np.abs(fin).max())
    assert st.g_min == float(F32(np.abs(fin).sum() / g.size))
    tail = np.abs(fin)[np.abs(fin).astype(F32) > F32(st.g_min)]
    assert st.n_tail == tail.size
    assert math.isclose(st.sum_log_tail, np.log(tail / np.float64(F32(st.g_min))).sum(), rel_tol=1e-11)
    st2 = orc.stats(g, g_min=2e-3)
    assert st2.g_min == float(F32(2e-3)) and st2.n_tail == int((np.abs(fin).astype(F32) > F32(2e-3)).sum())
    st3 = orc.stats(g, kappa=2.0)
    assert math.isclose(st3.g_min, 2 * st.g_min, rel_tol=1e-6)


def test_pow2_floor_is_the_power_of_two_below(orc):
    """The power-of-two threshold rule: pinned to 2^floor(log2 x) in float64 and to the bit pattern
    (mantissa cleared); exact at powers of two, just below them, and at the edges of the normal range."""
    rng = np.random.default_rng(12)
    xs = np.exp(rng.uniform(np.log(1e-37), np.log(3e38), 2000)).astype(F32)
    for x in xs:
        want = 2.0 ** math.floor(math.log2(float(x)))
        assert orc.pow2_floor(float(x)) == want
        assert orc.pow2_floor(float(x)) == float((np.array([x]).view(np.uint32) & np.uint32(0xFF800000)).view(F32)[0])
    for e in (-126, -20, -1, 0, 1, 30, 127):
        p2 = float(F32(2.0) ** e)
        assert orc.pow2_floor(p2) == p2
        assert orc.pow2_floor(float(np.nextafter(F32(p2), F32(np.inf)))) == p2
        if e > -126:
            assert orc.pow2_floor(float(np.nextafter(F32(p2), F32(0)))) == p2 / 2
    tiny = float(np.nextafter(F32(2.0) ** -126, F32(0)))            # largest subnormal: no tail
    assert orc.pow2_floor(tiny) == 0.0 and orc.pow2_floor(0.0) == 0.0 and orc.pow2_floor(1e-45) == 0.0
    assert orc.pow2_floor(float("inf")) == float("inf")


def test_stats_under_the_power_of_two_rule(orc):
    rng = np.random.default_rng(13)
    for scale, kappa in ((1e-3, 1.0), (1e-3, 2.5), (3.0, 1.0), (1e-30, 1.0)):
        g = (rng.standard_t(3.0, 50_001) * scale).astype(F32)
        g[[3, 9]] = [np.nan, -np.inf]
        plain = orc.stats(g, kappa=kappa)
        st = orc.stats_pow2(g, kappa=kappa)
        assert st.g_min <= plain.g_min < 2 * st.g_min and math.frexp(st.g_min)[0] == 0.5
        assert (st.sum_abs, st.sum_sq, st.max_abs, st.n_nonfinite) == (plain.sum_abs, plain.sum_sq, plain.max_abs, plain.n_nonfinite)
        fin = np.abs(g[np.isfinite(g)])
        tail = fin[fin > F32(st.g_min)].astype(np.float64)
        assert st.n_tail == tail.size >= plain.n_tail
        assert math.isclose(st.sum_log_tail, np.log(tail / st.g_min).sum(), rel_tol=1e-11)
    z = orc.stats_pow2(np.zeros(100, dtype=F32))
    assert z.g_min == 0.0 and z.n_tail == 0 and z.sum_log_tail == 0.0


def test_params_domain_errors(orc):
    st = orc.Stats(d=1000, n_tail=200, n_nonfinite=0, sum_abs=1.0, sum_sq=1.0, sum_log_tail=100.0,
                   max_abs=1.0, g_min=1e-3)
    for bad_gamma in (2.0, 1.5, float("inf")):
        with pytest.raises(orc.OracleError) as e:
            orc.params(st, 8, orc.UNIFORM, gamma=bad_gamma)
        assert e.value.code == orc.ERR_DOMAIN
    with pytest.raises(orc.OracleError):
        orc.params(st, 5, orc.UNIFORM, gamma=3.0)            # levels must be a power of two <= 16
    st0 = orc.Stats(d=1000, n_tail=0, n_nonfinite=0, sum_abs=1.0, sum_sq=1.0, sum_log_tail=0.0,
                    max_abs=1.0, g_min=1e-3)
    with pytest.raises(orc.OracleError):
        orc.params(st0, 8, orc.UNIFORM, gamma=3.0)           # no tail mass: rho = 0
    p = orc.params(st, 8, orc.UNIFORM, gamma=3.0, alpha_rule=orc.ALPHA_USER, alpha_user=0.25)
    assert p.alpha == 0.25
    pc = orc.params(st, 8, orc.UNIFORM, gamma=3.0, alpha_rule=orc.ALPHA_CLOSED)
    assert math.isclose(pc.alpha, 1e-3 * (2 * 0.1 * 49 / 1.0) ** 0.5, rel_tol=1e-6)


# ------------------------------------------------------------------ the optimum on data
@pytest.mark.parametrize("gamma,s", [(3.5, 7), (4.0, 7), (4.5, 15)])
def test_alpha_grid_search_on_samples(orc, gamma, s):
    """Brute-force alpha grid on samples drawn from the model: the error the paper minimises
    (Lemma 1's |Delta|^2/4 bound for the variance + the truncation bias) is smallest at the
    boxed alpha; the exact variance (Delta^2/6 at high rate) moves the empirical optimum to about
    alpha* (3/2)^(1/(gamma-1)), which is the expected consequence of minimising the bound."""
    rng = np.random.default_rng(100 + s)
    d, gm, rho = 300_000, 1e-3, 0.1
    g = _pareto_symmetric(rng, d, gm, rho, gamma).astype(np.float64)
    m = orc.Model(gm, rho, gamma)
    a_star, _, _ = orc.alpha_fixed_point(m, s, orc.UNIFORM)
    grid = a_star * np.exp(np.linspace(-0.7, 0.9, 81))
    absg = np.abs(g)

    def errors(alpha):
        step = 2 * alpha / s
        t = np.clip(g, -alpha, alpha)
        frac = np.mod((t + alpha) / step, 1.0)
        bias = np.mean(np.maximum(absg - alpha, 0) ** 2)
        inside = np.mean(absg <= alpha)
        return inside * step ** 2 / 4 + bias, np.mean(frac * (1 - frac)) * step ** 2 + bias

    e = np.array([errors(a) for a in grid])
    a_bound, a_exact = grid[e[:, 0].argmin()], grid[e[:, 1].argmin()]
    assert abs(math.log(a_bound / a_star)) < 0.10
    assert abs(math.log(a_exact / (a_star * 1.5 ** (1 / (gamma - 1))))) < 0.12


def test_no_truncation_baselines_use_the_full_range(orc):
    """QSGD / NQSGD of Section 5: the same quantizers without truncation, i.e. alpha = max|g|: no
    element is clipped and the largest element is reproduced exactly."""
    rng = np.random.default_rng(21)
    g = (rng.standard_t(2.5, 50_000) * 1e-3).astype(F32)
    st = orc.stats(g)
    for mode in (orc.UNIFORM, orc.NONUNIFORM):
        p = orc.params(st, 8, mode, gamma=3.0, alpha_rule=orc.ALPHA_MAXABS)
        assert p.alpha == st.max_abs and p.flags == 0
        lv = p.levels_np()
        assert lv[0] == -st.max_abs and lv[-1] == st.max_abs and np.all(np.diff(lv) > 0)
        for x in g[:2000]:
            assert orc.decision(p, float(x))[0] == float(x)          # T_alpha is the identity
        j = int(np.argmax(np.abs(g)))
        code = orc.code_from_bits(p, float(g[j]), 12345)
        assert lv[code] == g[j]
        # and it is a much coarser quantizer than the truncated one for a heavy tail
        pt = orc.params(st, 8, mode, gamma=3.0)
        assert p.alpha > 3 * pt.alpha
