"""What the 2^-16 resolution of the round-up probability costs at workload level (Lemma 1 is exact only for
probabilities that are multiples of 2^-16).

The oracle rounds an element up with probability T / 2^16, T = rint(p * 2^16), where p is the exact position
of the truncated value inside its interval.  So E[Q(g)] = l_k + (T / 2^16) |Delta_k| differs from the truncated
value by up to |Delta_k| 2^-17 (plus the fp32 rounding of p itself), and that deviation is deterministic for a
given value: it does not average out over workers or rounds the way the quantization noise does, unless the
values themselves change.  This test computes the EXACT expectation (no sampling) from the oracle's (k, T) on
inputs shaped like the benchmark workloads, including those where alpha = max|g| makes |Delta| huge compared
with a typical element, and states what the aggregate of N workers sees.
"""
import math

import numpy as np
import pytest
import torch

F32 = np.float32


def _rows(gamma, scale, d, n, seed, outliers=False, bf16=False):
    from paper_2402_01798_b200 import inputs
    rows = []
    for i in range(n):
        t = inputs.powerlaw_gradient(d, gamma, scale, seed + i, "cpu", torch.bfloat16 if bf16 else torch.float32,
                                     0.01 if outliers else 0.0, 100.0)
        rows.append(t.float().numpy())
    return rows


def _exact_moments(orc, p, g):
    """Per element: truncated value, exact mean and variance of the quantizer's output, interval width."""
    lv = p.levels_np().astype(np.float64)
    t = np.empty(g.size); mean = np.empty(g.size); var = np.empty(g.size); width = np.empty(g.size)
    for j, x in enumerate(g):
        tj, k, _, T = orc.decision(p, float(x))
        up = min(T, 65536) / 65536.0
        w = lv[k + 1] - lv[k]
        t[j], mean[j], var[j], width[j] = tj, lv[k] + up * w, up * (1.0 - up) * w * w, w
    return t, mean, var, width


CASES = [
    # name, gamma, scale, levels, mode, alpha rule, outliers, bf16
    ("config 1: uniform L4", 3.0, 1e-3, 4, "uniform", "fixed", False, False),
    ("config 3: non-uniform L16", 3.0, 5e-4, 16, "nonuniform", "fixed", False, False),
    ("config 4: bf16, outliers, gamma 2.2, non-uniform L16 (alpha capped at max|g|)", 2.2, 1e-4, 16, "nonuniform", "fixed", True, True),
    ("config 4: bf16, outliers, gamma 2.2, uniform L16", 2.2, 1e-4, 16, "uniform", "fixed", True, True),
    ("no truncation (alpha = max|g|), uniform L16", 3.0, 5e-4, 16, "uniform", "maxabs", False, False),
    ("no truncation (alpha = max|g|), non-uniform L16", 3.0, 5e-4, 16, "nonuniform", "maxabs", True, False),
    # a row of 124 M elements with gamma = 2.2 and 100x outliers has max|g| near 5e8 scale: plant that value, so that
    # |Delta| 2^-17 exceeds a typical element as it does at full size
    ("config 4 at full-size range: alpha = max|g| = 5e8 scale planted, non-uniform L16", 2.2, 1e-4, 16, "nonuniform", "fixed", True, True),
    ("config 4 at full-size range: alpha = max|g| = 5e8 scale planted, uniform L16", 2.2, 1e-4, 16, "uniform", "maxabs", True, True),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_bias_from_sixteen_bit_probabilities(orc, case, capsys):
    name, gamma, scale, L, mode, rule, outliers, bf16 = case
    d, n = 12_000, 4
    rows = _rows(gamma, scale, d, n, seed=31, outliers=outliers, bf16=bf16)
    m = orc.NONUNIFORM if mode == "nonuniform" else orc.UNIFORM
    bias_sum = np.zeros(d); var_sum = np.zeros(d); t_sum = np.zeros(d); worst = 0.0; dead = 0
    for g in rows:
        st = orc.stats(g)
        if "planted" in name:      # the sample's own tail statistics, alpha where a full-size row's maximum lies
            p = orc.build_table(orc.Model(st.g_min, st.n_tail / (2.0 * st.d), gamma), L, m, 5e8 * scale)
            g = g.copy(); g[17] = F32(5e8 * scale)
        else:
            p = orc.params(st, L, m, gamma, orc.ALPHA_MAXABS if rule == "maxabs" else orc.ALPHA_FIXED_POINT)
        if "capped" in name:
            assert p.flags & orc.FLAG_ALPHA_CAPPED
        t, mean, var, width = _exact_moments(orc, p, g)
        b = mean - t
        # per element: half a step of the 2^-16 grid, plus the fp32 rounding of p (a few ulp of the index x <= L)
        assert np.all(np.abs(b) <= width * (2.0 ** -17 + L * 2.0 ** -22))
        worst = max(worst, float(np.max(np.abs(b) / width)))
        dead += int(np.sum((var == 0) & (np.abs(b) > 0)))
        bias_sum += b; var_sum += var; t_sum += t
    keep = np.ones(d, dtype=bool)
    if "planted" in name:
        keep[17] = False                         # the norms below describe the ordinary elements
    agg_bias = (bias_sum / n)[keep]              # bias of the N-worker mean, per element
    agg_std = (np.sqrt(var_sum) / n)[keep]       # its quantization standard deviation
    t_sum = t_sum[keep]
    ratio_l2 = float(np.linalg.norm(agg_bias) / np.linalg.norm(agg_std))
    ratio_signal = float(np.linalg.norm(agg_bias) / np.linalg.norm(t_sum / n))     # against the truncated mean gradient itself
    mean_bias = float(np.mean(agg_bias)); mean_std = float(np.mean(agg_std))
    # The deviation is zero-mean across elements and five orders of magnitude below the noise of one round:
    assert ratio_l2 < 2e-5
    assert abs(mean_bias) < 3e-6 * mean_std
    # rounds of IDENTICAL gradients before the accumulated deviation reaches the accumulated noise: (1 / ratio)^2
    assert (1.0 / ratio_l2) ** 2 > 2e9
    with capsys.disabled():
        print(f"\n[R10] {name}: worst |bias|/|Delta| = {worst:.3e} (2^-17 = {2.0 ** -17:.3e}); ||bias|| / ||std|| of the "
              f"{n}-worker mean = {ratio_l2:.2e}; mean bias / mean std = {mean_bias / mean_std:+.1e}; "
              f"||bias|| / ||mean truncated gradient|| = {ratio_signal:.2e}; "
              f"elements rounded deterministically off their value: {dead} of {n * d}")
