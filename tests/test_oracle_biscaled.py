"""Pins for the oracle's truncated BiScaled quantizer (Appendix, "Truncated BiScaled Quantization").

As for the other parameter pins, nothing compares the oracle with itself: Q_B, the densities and
the error term are rebuilt from their defining integrals by quadrature, k* and the split
(s_alpha, s_beta) by brute force.
"""
import math

import numpy as np
import pytest
from scipy import integrate

F32 = np.float32
MODELS = [(1.0, 0.10, 4.0), (1e-3, 0.06, 3.5), (2e-4, 0.15, 5.0), (1e-3, 0.12, 3.2), (1e-3, 0.10, 3.0), (1e-3, 0.14, 2.5)]


def _quad(f, a, b, **kw):
    return integrate.quad(f, a, b, limit=400, epsabs=0, epsrel=1e-11, **kw)[0]


def _mass(orc, m, lo, hi):
    """2 * integral of the model density over [lo, hi] (0 <= lo < hi), by quadrature."""
    pts = [m.g_min] if lo < m.g_min < hi else None
    return 2 * _quad(lambda g: orc.model_fn("model_pdf", m, g), lo, hi, points=pts)


def _qb_by_definition(orc, m, alpha, k):
    inner, outer = _mass(orc, m, 0.0, k * alpha) if k > 0 else 0.0, _mass(orc, m, k * alpha, alpha) if k < 1 else 0.0
    return (outer ** (1 / 3) * (1 - k) ** (2 / 3) + inner ** (1 / 3) * k ** (2 / 3)) ** 3


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
def test_QB_is_its_definition_and_kstar_minimises_it(orc, gm, rho, gamma):
    m = orc.Model(gm, rho, gamma)
    for alpha in (1.5 * gm, 4.0 * gm, 25.0 * gm):
        for k in (0.0, 0.07, 0.3, 0.62, 0.95, 1.0):
            assert math.isclose(orc.model_fn("model_QB", m, alpha, k), _qb_by_definition(orc, m, alpha, k), rel_tol=1e-8)
        ks = orc.biscaled_kstar(m, alpha)
        grid = np.linspace(0.0, 1.0, 4001)
        vals = np.array([orc.model_fn("model_QB", m, alpha, float(k)) for k in grid])     # value checked above
        assert abs(ks - grid[vals.argmin()]) <= 2.5e-4 + 1e-3 * (vals.max() - vals.min() < 1e-9)
        qb = orc.model_fn("model_QB", m, alpha, ks)
        assert qb <= vals.min() * (1 + 1e-9)
        # k = 1 is the uniform quantizer; the cube-root density is the best of all (Hoelder)
        assert math.isclose(orc.model_fn("model_QB", m, alpha, 1.0), orc.model_fn("model_QU", m, alpha), rel_tol=1e-12)
        assert orc.model_fn("model_QN", m, alpha) <= qb * (1 + 1e-9) <= orc.model_fn("model_QU", m, alpha) * (1 + 1e-9) <= 1 + 1e-9


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
@pytest.mark.parametrize("s", [7, 15])
def test_boxed_density_integrates_to_s_and_gives_the_error_term(orc, gm, rho, gamma, s):
    """lambda integrates to s; (1/4) int p / lambda^2 over [-alpha, alpha] equals Q_B alpha^2 / s^2
    (the first term of the Appendix error equation); s_alpha, s_beta follow the Appendix formulas and
    are the best split of s for that k."""
    m = orc.Model(gm, rho, gamma)
    pdf = lambda g: orc.model_fn("model_pdf", m, g)
    alpha = 9.0 * gm
    k, lam_in, lam_out = orc.biscaled_density(m, alpha, s)
    beta = k * alpha
    assert math.isclose(2 * beta * lam_in + 2 * (alpha - beta) * lam_out, s, rel_tol=1e-12)
    p1, p2 = _mass(orc, m, 0, beta) / (2 * beta), _mass(orc, m, beta, alpha) / (2 * (alpha - beta))
    assert math.isclose(lam_in / lam_out, (p1 / p2) ** (1 / 3), rel_tol=1e-8)
    pts_in = [gm] if gm < beta else None
    pts_out = [gm] if beta < gm < alpha else None
    var = 0.25 * 2 * (_quad(lambda g: pdf(g) / lam_in ** 2, 0, beta, points=pts_in)
                      + _quad(lambda g: pdf(g) / lam_out ** 2, beta, alpha, points=pts_out))
    assert math.isclose(var, orc.model_fn("model_QB", m, alpha, k) * alpha ** 2 / s ** 2, rel_tol=1e-7)
    if gamma > 3:
        bias = orc.model_fn("truncation_bias", m, alpha)
        assert math.isclose(orc.model_fn("etq_biscaled", m, alpha, s), var + bias, rel_tol=1e-7)
    # Appendix: s_beta = p1^(1/3) k / (p2^(1/3)(1-k) + p1^(1/3) k) * s, s_alpha = the rest
    s_beta, s_alpha = 2 * beta * lam_in, 2 * (alpha - beta) * lam_out
    c1, c2 = p1 ** (1 / 3), p2 ** (1 / 3)
    assert math.isclose(s_beta, c1 * k / (c2 * (1 - k) + c1 * k) * s, rel_tol=1e-8)
    # brute force over the split: 2 p1 beta^3 / s_b^2 + 2 p2 (alpha - beta)^3 / s_a^2 with s_a + s_b = s
    cost = lambda sb: 2 * p1 * beta ** 3 / sb ** 2 + 2 * p2 * (alpha - beta) ** 3 / (s - sb) ** 2
    grid = np.linspace(0.02 * s, 0.98 * s, 20001)
    assert abs(grid[np.argmin(cost(grid))] - s_beta) <= 2 * (grid[1] - grid[0])
    assert math.isclose(cost(s_beta), var, rel_tol=1e-7)      # Appendix, expression before the error equation


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
@pytest.mark.parametrize("L", [4, 8, 16])
def test_biscaled_levels_are_one_cell_of_density_apart(orc, gm, rho, gamma, L):
    m = orc.Model(gm, rho, gamma)
    s = L - 1
    for alpha in (2.0 * gm, 12.0 * gm):
        p = orc.build_table(m, L, orc.BISCALED, alpha)
        lv = p.levels_np().astype(np.float64)
        a = float(p.alpha)
        k, lam_in, lam_out = orc.biscaled_density(m, a, s)
        beta = k * a
        lam = lambda g: lam_in if abs(g) <= beta else lam_out
        assert lv[0] == -a and lv[-1] == a and np.all(np.diff(lv) > 0) and np.array_equal(lv, -lv[::-1])
        for j in range(s):
            lo, hi = lv[j], lv[j + 1]
            pts = [x for x in (-beta, beta) if lo < x < hi] or None
            assert math.isclose(_quad(lam, lo, hi, points=pts), 1.0, rel_tol=3e-6), (alpha, j)
        # two step sizes only: inside and outside +-beta (cells that straddle beta excepted)
        widths = np.diff(lv)
        inside = [w for j, w in enumerate(widths) if abs(lv[j]) <= beta and abs(lv[j + 1]) <= beta]
        outside = [w for j, w in enumerate(widths) if abs(lv[j]) >= beta and abs(lv[j + 1]) >= beta]
        for grp, lamv in ((inside, lam_in), (outside, lam_out)):
            for w in grp:
                assert math.isclose(w, 1 / lamv, rel_tol=2e-5)


@pytest.mark.parametrize("gm,rho,gamma", MODELS)
@pytest.mark.parametrize("s", [3, 7, 15])
def test_biscaled_alpha_solves_the_boxed_equation(orc, gm, rho, gamma, s):
    m = orc.Model(gm, rho, gamma)
    a, iters, capped = orc.alpha_fixed_point(m, s, orc.BISCALED)
    assert not capped and iters < 10000
    ks = orc.biscaled_kstar(m, a)
    qb = _qb_by_definition(orc, m, a, ks)
    assert math.isclose(a, gm * (2 * rho * s * s / ((gamma - 2) * qb)) ** (1 / (gamma - 1)), rel_tol=1e-7)
    au, _, _ = orc.alpha_fixed_point(m, s, orc.UNIFORM)
    an, _, _ = orc.alpha_fixed_point(m, s, orc.NONUNIFORM)
    assert au * (1 - 1e-9) <= a <= an * (1 + 1e-9)          # between the uniform and the cube-root quantizer
    if gamma > 3 and a > gm:
        e = orc.model_fn("etq_biscaled", m, a, s)
        assert math.isclose(e, orc.model_fn("etq_theorem", m, qb, s), rel_tol=1e-6)      # Appendix theorem (TBQSGD)
        assert orc.model_fn("etq_nonuniform", m, an, s) * (1 - 1e-9) <= e <= orc.model_fn("etq_uniform", m, au, s) * (1 + 1e-9)


def test_biscaled_params_from_statistics_and_quantizer_is_unbiased(orc):
    rng = np.random.default_rng(8)
    g = (rng.standard_t(3.0, 100_000) * 1e-3).astype(F32)
    st = orc.stats(g)
    p = orc.params(st, 8, orc.BISCALED, gamma=3.5)
    assert p.mode == orc.BISCALED and p.bits == 3 and p.alpha > st.g_min
    lv = p.levels_np().astype(np.float64)
    for x in (0.3 * p.alpha, -0.77 * p.alpha, 1e-5, float(lv[2])):
        t, k, pr, T = orc.decision(p, x)
        assert lv[k] <= t <= lv[k + 1]
        mean = lv[k] + (lv[k + 1] - lv[k]) * min(T, 65536) / 65536.0
        assert abs(mean - t) <= (lv[k + 1] - lv[k]) * (2.0 ** -17 + 4e-6)
