"""Pins for the oracle's truncation + stochastic quantizer (Section 3.1, Lemma 1).

Nothing here compares the oracle with itself: expectations and variances are obtained by
ENUMERATING all 2^16 values of the random slot (so they are exact, not sampled), interval
indices come from NumPy's binary search, truncation from ``np.clip``, and the Monte-Carlo
and exhaustive-outcome tests use only the definition of the quantizer in the paper.
"""
import itertools
import math

import numpy as np
import pytest

F32 = np.float32


def _model(orc, g_min=1e-3, rho=0.12, gamma=3.0):
    return orc.Model(g_min, rho, gamma)


def _tables(orc):
    """A spread of codebooks: uniform and non-uniform, 2/3/4 bits."""
    out = []
    for L in (4, 8, 16):
        out.append(orc.build_table(_model(orc), L, orc.UNIFORM, 0.004))
        out.append(orc.build_table(_model(orc), L, orc.NONUNIFORM, 0.03))
    out.append(orc.build_table(_model(orc, gamma=4.5), 16, orc.NONUNIFORM, 0.0021))
    out.append(orc.build_table(_model(orc), 2, orc.UNIFORM, 0.5))
    return out


def _probe_values(p, rng, n=60):
    a = p.alpha
    lv = p.levels_np()
    vals = list(rng.uniform(-1.3 * a, 1.3 * a, n).astype(F32))
    vals += list(lv)                                   # exactly on codebook points
    vals += [np.nextafter(x, F32(np.inf)) for x in lv[:-1]]
    vals += [np.nextafter(x, F32(-np.inf)) for x in lv[1:]]
    vals += [F32(0.0), F32(-0.0), F32(a), F32(-a), F32(10 * a), F32(-10 * a),
             F32(np.inf), F32(-np.inf), F32(1e-30), F32(-1e-30)]
    return [float(v) for v in vals]


def test_truncation_is_clip(orc):
    """T_alpha[g] = g inside [-alpha, alpha], sgn(g) alpha outside (truncation equation)."""
    rng = np.random.default_rng(0)
    for p in _tables(orc):
        for g in _probe_values(p, rng):
            t, _, _, _ = orc.decision(p, g)
            assert t == float(np.clip(F32(g), F32(-p.alpha), F32(p.alpha)))
        t, k, pr, T = orc.decision(p, float("nan"))    # documented: NaN is sent to -alpha, code 0
        assert t == -p.alpha and k == 0 and T == 0


def test_interval_index_matches_binary_search(orc):
    """g in Delta_k = [l_{k-1}, l_k] (paper's 1-based k): the oracle's 0-based interval index equals
    NumPy's searchsorted on the codebook (values on a point belong to the interval they start)."""
    rng = np.random.default_rng(1)
    for p in _tables(orc):
        lv = p.levels_np()
        s = p.num_levels - 1
        for g in _probe_values(p, rng):
            t, k, pr, T = orc.decision(p, g)
            want = int(np.clip(np.searchsorted(lv, F32(t), side="right") - 1, 0, s - 1))
            if p.mode == orc.UNIFORM:
                # the uniform index is computed arithmetically; within rounding of a codebook
                # point it may name the neighbouring interval with p_r ~ 0 or ~ 1 (same value)
                near = np.min(np.abs(lv.astype(np.float64) - t)) <= 4e-7 * p.alpha * s
                if near and k != want:
                    assert abs(k - want) == 1
                    continue
            assert k == want, (p.mode, p.num_levels, g)
            assert lv[k] <= t <= lv[k + 1] or p.mode == orc.UNIFORM


def test_round_up_probability_is_linear_in_cell(orc):
    """p_r = (g - l_{k-1}) / |Delta_k| (quantizer equation), to fp32 rounding."""
    rng = np.random.default_rng(2)
    for p in _tables(orc):
        lv = p.levels_np().astype(np.float64)
        for g in _probe_values(p, rng):
            t, k, pr, T = orc.decision(p, g)
            want = (t - lv[k]) / (lv[k + 1] - lv[k])
            assert abs(pr - want) <= 3e-6, (p.mode, p.num_levels, g, pr, want)
            assert T == int(np.rint(F32(pr) * F32(65536.0)))
            assert 0 <= T <= 65536 + 1


def test_exact_expectation_and_variance_by_enumerating_the_random_slot(orc):
    """Lemma 1: E Q[g] = g and E (Q[g]-g)^2 = (g-l_{k-1})(l_k-g) <= |Delta_k|^2/4.

    The 16 random bits are enumerated exhaustively, so the expectation is exact; the only
    departure from g is the 2^-16 granularity of the probability (at most |Delta|*2^-17)
    plus fp32 rounding of p_r."""
    rng = np.random.default_rng(3)
    all_r = range(65536)
    for p in _tables(orc)[:6:2] + _tables(orc)[1:6:2]:
        lv = p.levels_np().astype(np.float64)
        for g in _probe_values(p, rng, n=6)[:14]:
            t, k, pr, T = orc.decision(p, g)
            codes = np.array([orc.code_from_bits(p, g, r) for r in all_r])
            assert set(np.unique(codes)) <= {k, k + 1}
            n_up = int((codes == k + 1).sum())
            assert n_up == min(T, 65536)               # exactly T of the 65536 slots round up
            assert np.all(codes[:n_up] == k + 1) and np.all(codes[n_up:] == k)
            width = lv[k + 1] - lv[k]
            mean = lv[k] + width * n_up / 65536.0
            assert abs(mean - t) <= width * (2.0 ** -17 + 4e-6)
            var = (n_up / 65536.0) * (lv[k + 1] - t) ** 2 + (1 - n_up / 65536.0) * (lv[k] - t) ** 2
            assert abs(var - (t - lv[k]) * (lv[k + 1] - t)) <= width ** 2 * 1e-4
            assert var <= width ** 2 / 4 * (1 + 1e-6)


def test_top_and_bottom_of_range_are_deterministic(orc):
    """|g| >= alpha is truncated onto a codebook point, which is reproduced exactly (R11)."""
    for p in _tables(orc):
        s = p.num_levels - 1
        for r in (0, 1, 32768, 65535):
            assert orc.code_from_bits(p, p.alpha, r) == s
            assert orc.code_from_bits(p, 7 * p.alpha, r) == s
            assert orc.code_from_bits(p, float("inf"), r) == s
            assert orc.code_from_bits(p, -p.alpha, r) == 0
            assert orc.code_from_bits(p, -7 * p.alpha, r) == 0
            assert orc.code_from_bits(p, float("-inf"), r) == 0
        if p.mode == orc.NONUNIFORM:                   # interior codebook points are fixed points too
            for k, l in enumerate(p.levels_np()):
                for r in (0, 65535):
                    assert orc.code_from_bits(p, float(l), r) == k


def test_high_rate_cell_average_is_delta_squared_over_six(orc):
    """Proof of Lemma 1, step (a): with a flat density inside a cell, the mean of the exact
    per-element variance p_r (1 - p_r) |Delta|^2 is |Delta|^2 / 6."""
    p = orc.build_table(_model(orc), 8, orc.NONUNIFORM, 0.02)
    lv = p.levels_np().astype(np.float64)
    for k in (0, 3, 6):
        ts = np.linspace(lv[k], lv[k + 1], 4001)[1:-1]
        prs = np.array([orc.decision(p, float(F32(t)))[2] for t in ts], dtype=np.float64)
        width = lv[k + 1] - lv[k]
        assert abs(np.mean(prs * (1 - prs)) * width ** 2 - width ** 2 / 6) <= 2e-3 * width ** 2


def test_unbiased_by_monte_carlo_over_seeds(orc):
    """E Q[T_alpha g] = clip(g, -alpha, alpha), sampled through the full seeded path
    (Philox counter scheme included), for uniform and non-uniform codebooks."""
    rng = np.random.default_rng(4)
    d, n_seeds = 256, 1500
    for p in (orc.build_table(_model(orc), 8, orc.UNIFORM, 0.004),
              orc.build_table(_model(orc), 16, orc.NONUNIFORM, 0.03)):
        g = (rng.standard_t(2.5, d) * 1e-3).astype(F32)
        lv = p.levels_np().astype(np.float64)
        acc = np.zeros(d)
        acc2 = np.zeros(d)
        for sd in range(n_seeds):
            v = lv[orc.quantize(g, p, seed=1000 + sd, worker=3)]
            acc += v
            acc2 += v * v
        mean = acc / n_seeds
        var = np.maximum(acc2 / n_seeds - mean ** 2, 0)
        clip = np.clip(g.astype(np.float64), -p.alpha, p.alpha)
        widths = np.diff(lv).max()
        z = np.abs(mean - clip) / np.sqrt(var / n_seeds + (1e-6 * widths) ** 2)
        assert z.max() < 5.0 and np.mean(z > 3.0) < 0.02
        # and the sampled variance respects Lemma 1's per-element bound
        assert np.all(var <= (widths ** 2 / 4) * 1.2)


@pytest.mark.parametrize("d", [1, 3, 9, 16])
def test_exhaustive_outcomes_small_d(orc, d):
    """For d <= 16 every element has at most two reachable codes; all 2^d outcome vectors are
    enumerated with their exact probabilities (T/2^16 per element, independent slots):
    probabilities sum to one, the expectation is the truncated vector, and every seeded run
    of the full path lands on a reachable outcome."""
    rng = np.random.default_rng(10 + d)
    p = orc.build_table(_model(orc), 4, orc.NONUNIFORM, 0.01)
    lv = p.levels_np().astype(np.float64)
    g = (rng.standard_t(3.0, d) * 2e-3).astype(F32)
    dec = [orc.decision(p, float(x)) for x in g]
    ks = np.array([k for _, k, _, _ in dec])
    pu = np.array([min(T, 65536) / 65536.0 for _, _, _, T in dec])
    total, expect = 0.0, np.zeros(d)
    for ups in itertools.product((0, 1), repeat=d):
        ups = np.array(ups)
        pr = np.prod(np.where(ups == 1, pu, 1 - pu))
        total += pr
        expect += pr * lv[ks + ups]
    assert abs(total - 1.0) < 1e-12
    t = np.array([tt for tt, _, _, _ in dec], dtype=np.float64)
    widths = lv[ks + 1] - lv[ks]
    assert np.all(np.abs(expect - t) <= widths * (2.0 ** -17 + 4e-6))
    for sd in range(200):
        codes = orc.quantize(g, p, seed=sd, worker=0).astype(np.int64)
        ups = codes - ks
        assert np.all((ups == 0) | (ups == 1))
        assert np.all((pu > 0) | (ups == 0)) and np.all((pu < 1) | (ups == 1))


def test_joint_outcome_frequencies_match_product_law(orc):
    """Slots of one Philox block are used as independent draws: for d = 3 the 8 joint outcomes
    occur with the product of the per-element probabilities (chi-square over many seeds)."""
    p = orc.build_table(_model(orc), 4, orc.UNIFORM, 0.004)
    lv = p.levels_np().astype(np.float64)
    g = np.array([0.3 * lv[1] + 0.7 * lv[2], 0.5 * lv[0] + 0.5 * lv[1], 0.8 * lv[2] + 0.2 * lv[3]], dtype=F32)
    dec = [orc.decision(p, float(x)) for x in g]
    ks = np.array([k for _, k, _, _ in dec])
    pu = np.array([T / 65536.0 for _, _, _, T in dec])
    n = 8000
    counts = np.zeros(8)
    for sd in range(n):
        ups = orc.quantize(g, p, seed=sd * 7919 + 1, worker=2).astype(np.int64) - ks
        counts[ups[0] * 4 + ups[1] * 2 + ups[2]] += 1
    exp = np.array([np.prod(np.where(np.array(u) == 1, pu, 1 - pu)) for u in itertools.product((0, 1), repeat=3)]) * n
    chi2 = ((counts - exp) ** 2 / exp).sum()
    assert chi2 < 7 + 6 * math.sqrt(14)


def test_code_at_is_quantize_elementwise(orc):
    """The per-element entry point used for sampled full-size parity agrees with the vector path."""
    rng = np.random.default_rng(5)
    p = orc.build_table(_model(orc), 8, orc.NONUNIFORM, 0.02)
    g = (rng.standard_t(2.5, 1000) * 1e-3).astype(F32)
    codes = orc.quantize(g, p, seed=99, worker=4)
    for j in (0, 1, 7, 8, 9, 511, 999):
        assert orc.code_at(p, float(g[j]), 99, 4, j) == codes[j]
