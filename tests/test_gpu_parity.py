"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle.

Chain of custody: every stage is compared on the SAME inputs.  The oracle is handed the very bytes
the GPU consumed (copied back) and, for the bit-exact stages, the library's own upstream outputs
(its g_min, its quantizer parameters); each upstream output is itself compared with the oracle's.

Bars: packed words / codes bit-exact; aggregated updates within 1e-6 relative per element (the
pinned arithmetic actually gives equality, which is asserted too); statistics: counts and max
exact, sums to the tolerance derived from the kernel's fp32-over-16-elements accumulation.
"""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

F32 = np.float32
# sums: 16 positive fp32 terms are added before going to fp64: relative error <= 15 * 2^-24 ~ 9e-7,
# plus 2^-24 for the square.  The logarithm uses the hardware lg2 approximation (absolute error about
# 2^-22 per term, terms of order one).
TOL_SUM = 2e-6
TOL_LOG = 5e-6


@pytest.fixture(scope="module")
def tq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_01798_b200 import binding
    binding.lib()                    # must be prebuilt and in-tree: no fallback
    return binding


def to_oracle_params(orc, p):
    q = orc.Params()
    for f in ("bits", "num_levels", "mode", "flags", "alpha", "inv_step", "gamma", "g_min", "rho", "iterations"):
        setattr(q, f, getattr(p, f))
    for k in range(16):
        q.levels[k] = p.levels[k]
        q.inv_width[k] = p.inv_width[k]
    return q


def host_f32(orc, t: torch.Tensor) -> np.ndarray:
    """The bytes the GPU consumed, as the fp32 values the method sees."""
    if t.dtype == torch.bfloat16:
        return orc.bf16_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.cpu().numpy()


def heavy_tailed(d, n, dtype, seed, scale=1e-3, gamma=3.0, device="cuda"):
    from paper_2402_01798_b200 import inputs
    stride = inputs.worker_stride(d, dtype)
    g = torch.zeros((n, stride), dtype=dtype, device=device)
    for i in range(n):
        if d:
            inputs.powerlaw_gradient(d, gamma, scale, seed + i, device, dtype, out=g[i, :d])
    return g


def salt_special_values(g, d, p):
    """Overwrite a few entries with the degenerate inputs the method has."""
    vals = [float("nan"), float("inf"), float("-inf"), p.alpha, -p.alpha, 0.0, -0.0,
            2 * p.alpha, -2 * p.alpha, 1e-38, 3e38] + [p.levels[k] for k in range(p.num_levels)]
    rng = np.random.default_rng(d)
    idx = rng.choice(d, size=min(d, len(vals)), replace=False)
    for i, v in zip(idx, vals):
        g[:, int(i)] = v


def lib_params_for(tq, g, d, L, mode, gamma, rule=None):
    st = tq.stats_to_host(tq.tq_stats(g, d))
    rule = tq.ALPHA_FIXED_POINT if rule is None else rule
    return st, [tq.tq_params(s, L, mode, gamma, rule) for s in st]


# ----------------------------------------------------------------------------------------- stats
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d,n", [(0, 1), (1, 1), (15, 2), (16, 1), (17, 3), (4099, 2), (100_003, 3), (3_000_000, 4)])
def test_stats_parity(tq, orc, d, n, dtype):
    g = heavy_tailed(d, n, dtype, seed=d + 1)
    if d > 40:
        g[:, 7] = float("nan"); g[:, 33] = float("inf"); g[0, 21] = float("-inf")
    for g_min_in in (0.0, 7e-4):
        for kappa in ((1.0, 2.5) if g_min_in == 0.0 else (1.0,)):
            got = tq.stats_to_host(tq.tq_stats(g, d, g_min=g_min_in, kappa=kappa))
            assert len(got) == n
            for i in range(n):
                x = host_f32(orc, g[i, :d])
                auto = orc.stats(x, g_min=g_min_in, kappa=kappa)          # oracle's own threshold
                s = got[i]
                assert s.d == d and s.n_nonfinite == auto.n_nonfinite and s.max_abs == auto.max_abs
                assert math.isclose(s.sum_abs, auto.sum_abs, rel_tol=TOL_SUM, abs_tol=0)
                assert math.isclose(s.sum_sq, auto.sum_sq, rel_tol=TOL_SUM, abs_tol=0)
                assert math.isclose(s.g_min, auto.g_min, rel_tol=TOL_SUM, abs_tol=0)
                if g_min_in > 0:
                    assert s.g_min == F32(g_min_in)
                ref = orc.stats(x, g_min=s.g_min) if s.g_min > 0 else auto   # tail part on the library's g_min
                assert s.n_tail == ref.n_tail
                assert math.isclose(s.sum_log_tail, ref.sum_log_tail, rel_tol=TOL_LOG, abs_tol=1e-9)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d,n", [(0, 1), (1, 1), (17, 3), (4099, 2), (100_003, 3), (3_000_000, 4)])
def test_stats_hinted_parity_and_hint_independence(tq, orc, d, n, dtype):
    """tq_stats_hinted against the oracle under the power-of-two threshold rule; the record must be the
    same bit for bit whether the tail came from the single pass (hint hit) or from the second kernel
    (no hint, stale hint)."""
    g = heavy_tailed(d, n, dtype, seed=d + 3)
    if d > 40:
        g[:, 7] = float("nan"); g[:, 33] = float("inf"); g[0, 21] = float("-inf")
    for kappa in (1.0, 2.5):
        hint = tq.new_gmin_hint(n)
        first = tq.tq_stats_hinted(g, hint, d, kappa=kappa).cpu().numpy().tobytes()       # no hint: second kernel
        h1 = tq.gmin_hint_to_host(hint)
        again = tq.tq_stats_hinted(g, hint, d, kappa=kappa).cpu().numpy().tobytes()       # hint from the same data
        h2 = tq.gmin_hint_to_host(hint)
        assert first == again
        got = tq.stats_to_host(torch.frombuffer(bytearray(again), dtype=torch.uint8))
        for i in range(n):
            x = host_f32(orc, g[i, :d])
            want = orc.stats_pow2(x, kappa=kappa)
            s = got[i]
            assert s.d == d and s.n_nonfinite == want.n_nonfinite and s.max_abs == want.max_abs
            assert math.isclose(s.sum_abs, want.sum_abs, rel_tol=TOL_SUM, abs_tol=0)
            assert math.isclose(s.sum_sq, want.sum_sq, rel_tol=TOL_SUM, abs_tol=0)
            level = F32(kappa * s.sum_abs / d) if d else F32(0)
            assert s.g_min == orc.pow2_floor(float(level))               # the rule, on the library's own mean
            assert math.isclose(h2[i][0], float(level), rel_tol=1e-6, abs_tol=0) and h2[i][0] == h1[i][0]
            assert h2[i][1] == 1 and h1[i][1] == (0 if s.g_min > 0 else 1)
            if s.g_min == want.g_min:                                     # same binade as the oracle's mean (always, bar ties)
                assert s.n_tail == want.n_tail
                assert math.isclose(s.sum_log_tail, want.sum_log_tail, rel_tol=TOL_LOG, abs_tol=1e-9)
        # a stale hint (mean moved by 8x): the second kernel runs again, same record
        hint2 = tq.new_gmin_hint(n)
        tq.tq_stats_hinted(g * 8 if dtype == torch.float32 else (g.float() * 8).to(dtype), hint2, d, kappa=kappa)
        stale = tq.tq_stats_hinted(g, hint2, d, kappa=kappa).cpu().numpy().tobytes()
        assert stale == first
        if d > 40:
            assert all(hit == 0 for _, hit in tq.gmin_hint_to_host(hint2))
        # a hint one binade off still hits: candidates are the two powers of two nearest to it
        hint3 = tq.new_gmin_hint(n)
        tq.tq_stats_hinted((g.float() * 1.3).to(dtype), hint3, d, kappa=kappa)
        near = tq.tq_stats_hinted(g, hint3, d, kappa=kappa).cpu().numpy().tobytes()
        assert near == first
        if d > 40:
            assert all(hit == 1 for _, hit in tq.gmin_hint_to_host(hint3))


def test_stats_hinted_degenerate_rows(tq, orc):
    """All-zero and all-non-finite rows: no threshold (g_min = 0), no tail, and the hint says so."""
    d = 5000
    g = torch.zeros((3, d), dtype=torch.float32, device="cuda")
    g[1, :] = float("nan")
    g[2, ::2] = float("inf")
    hint = tq.new_gmin_hint(3)
    for _ in range(2):
        st = tq.stats_to_host(tq.tq_stats_hinted(g, hint, d))
        for i, bad in enumerate((0, d, d // 2)):
            want = orc.stats_pow2(g[i].cpu().numpy())
            assert (st[i].g_min, st[i].n_tail, st[i].sum_log_tail, st[i].n_nonfinite) == (0.0, 0, 0.0, bad)
            assert (want.g_min, want.n_tail, want.n_nonfinite) == (0.0, 0, bad)
        assert all(hit == 1 for _, hit in tq.gmin_hint_to_host(hint))


def test_stats_is_deterministic_and_reuses_workspace(tq):
    g = heavy_tailed(1_000_003, 4, torch.float32, seed=3)
    ws = torch.empty(tq.tq_stats_workspace_bytes(4), dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)                                        # scratch contents need not be initialised
    a = tq.tq_stats(g, 1_000_003, workspace=ws).cpu()
    b = tq.tq_stats(g, 1_000_003, workspace=ws).cpu()
    c = tq.tq_stats(g, 1_000_003).cpu()
    assert torch.equal(a, b) and torch.equal(a, c)


# -------------------------------------------------------------------------------------- compress
SIZES = [1, 3, 8, 31, 32, 33, 127, 255, 256, 257, 8191, 8192, 8193, 100_003]


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_compress_bit_exact_ragged_sizes(tq, orc, bits, mode, dtype):
    L = 1 << bits
    for d in SIZES:
        n = 1 if d % 2 else 3
        g = heavy_tailed(d, n, dtype, seed=100 * bits + d)
        st = [orc.stats(host_f32(orc, g[i, :d]), g_min=5e-4) for i in range(n)]
        ps = []
        for i, s in enumerate(st):                        # parameters from the library's host code
            ls = tq.Stats(d=max(s.d, 1000), n_tail=max(s.n_tail, 100), n_nonfinite=0, sum_abs=s.sum_abs, sum_sq=s.sum_sq,
                          sum_log_tail=max(s.sum_log_tail, 50.0), max_abs=max(s.max_abs, 0.05), g_min=5e-4)
            ps.append(tq.tq_params(ls, L, mode, 3.0 + 0.25 * i))
        if d >= 64:
            salt_special_values(g, d, ps[0])
        seed, first = 0xC0FFEE123456789, 5
        words = tq.tq_packed_words(d, bits)
        packed = torch.full((n, words + 8), 0x5A5A5A5A, dtype=torch.int32, device="cuda")   # canary beyond the row
        tq.tq_compress(g, ps, seed, first, d=d, packed=packed)
        got = packed.cpu().numpy().view(np.uint32)
        for i in range(n):
            want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), seed, first + i)
            assert want.size == words
            assert np.array_equal(got[i, :words], want), (d, i)
            assert np.all(got[i, words:] == 0x5A5A5A5A)    # nothing written past the row's words


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_compress_tiled_copy_path_ragged_sizes(tq, orc, bits, mode, dtype):
    """Table-mode bf16 rows of 65536 elements and more go through the kernel that brings the gradient in by
    tiled copies (tiles of 8192 elements; fp32 rows and uniform mode keep the direct kernel and run here too):
    whole tiles, one run more or less, a partial last run, a last tile with a single run, several workers
    with a padded row stride; salted with NaN, Inf, levels."""
    L = 1 << bits
    for d, n in ((65_536, 2), (65_537, 1), (65_568, 3), (73_728, 1), (73_729, 2), (81_919, 1), (200_003, 3)):
        g = heavy_tailed(d, n, dtype, seed=7 * bits + d)
        ps = []
        for i in range(n):
            s = orc.stats(host_f32(orc, g[i, :d]), g_min=5e-4)
            ls = tq.Stats(d=s.d, n_tail=max(s.n_tail, 100), n_nonfinite=0, sum_abs=s.sum_abs, sum_sq=s.sum_sq,
                          sum_log_tail=max(s.sum_log_tail, 50.0), max_abs=max(s.max_abs, 0.05), g_min=5e-4)
            ps.append(tq.tq_params(ls, L, mode, 3.0 + 0.25 * i))
        salt_special_values(g, d, ps[0])
        seed, first = 0x1234ABCD5678, 3
        words = tq.tq_packed_words(d, bits)
        packed = torch.full((n, words + 8), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
        tq.tq_compress(g, ps, seed, first, d=d, packed=packed)
        got = packed.cpu().numpy().view(np.uint32)
        for i in range(n):
            want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), seed, first + i)
            assert np.array_equal(got[i, :words], want), (d, i)
            assert np.all(got[i, words:] == 0x5A5A5A5A)
    torch.cuda.synchronize()
    assert tq.tq_wait_expired_count() == 0


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("mode", [0, 1])
def test_compress_decision_table_path_ragged_sizes(tq, orc, bits, mode):
    """bf16 rows of 2^18 elements and more take the kernel that reads the decision (interval and threshold)
    from a per-block table indexed by the element's bit pattern: whole tiles, one element more, a partial
    last run, several workers with a padded stride and different quantizers; salted with NaN of both signs,
    Inf, +-alpha, zeros, subnormals and the levels themselves."""
    L = 1 << bits
    for d, n in ((262_144, 2), (262_145, 1), (262_176, 3), (270_337, 2), (300_003, 3)):
        g = heavy_tailed(d, n, torch.bfloat16, seed=13 * bits + d)
        ps = []
        for i in range(n):
            s = orc.stats(host_f32(orc, g[i, :d]), g_min=5e-4)
            ls = tq.Stats(d=s.d, n_tail=max(s.n_tail, 100), n_nonfinite=0, sum_abs=s.sum_abs, sum_sq=s.sum_sq,
                          sum_log_tail=max(s.sum_log_tail, 50.0), max_abs=max(s.max_abs, 0.05), g_min=5e-4)
            ps.append(tq.tq_params(ls, L, mode, 3.0 + 0.25 * i))
        salt_special_values(g, d, ps[0])
        g[:, 5] = -float("nan")
        g.view(torch.int16)[:, 6] = 0x7FFF                                               # NaN with the largest payload
        g.view(torch.int16)[:, 7] = -1                                                   # the same with the sign set
        g.view(torch.int16)[:, 8] = 1                                                    # smallest subnormal
        g.view(torch.int16)[:, 9] = -32767                                               # its negative
        seed, first = 0x9E3779B97F4A7C15, 2
        words = tq.tq_packed_words(d, bits)
        packed = torch.full((n, words + 8), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
        tq.tq_compress(g, ps, seed, first, d=d, packed=packed)
        got = packed.cpu().numpy().view(np.uint32)
        for i in range(n):
            want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), seed, first + i)
            assert np.array_equal(got[i, :words], want), (d, i)
            assert np.all(got[i, words:] == 0x5A5A5A5A)


def test_compress_decision_table_windows_and_fallback(tq, orc):
    """The table covers a window of 16, 32 or 64 binades below alpha.  Codebooks whose scale puts the window
    at the bottom of the exponent range, at its top, and whose central levels are too small for any window
    (the element-wise kernel then runs) all give the oracle's codes; so does alpha = max|g| (no truncation)."""
    d = 262_144 + 77
    books = [
        np.array([-1e-36, -3e-37, 2e-37, 1e-36], dtype=F32),                    # window reaches zero
        np.array([-3e30, -1e30, -1e29, 1e28, 2e29, 5e29, 2e30, 3e30], dtype=F32),   # window high in the exponent range
        np.array([-1.0, -1e-30, 1e-30, 1.0], dtype=F32),                         # no window: 100 binades between alpha and the centre
        np.concatenate([[-2e-3], np.linspace(-1e-7, 1e-7, 14), [2e-3]]).astype(F32),   # crowded at zero, 64 binades
        np.linspace(-0.75, 0.75, 16).astype(F32),
    ]
    for lv in books:
        p = tq.tq_params_from_levels([float(x) for x in lv])
        g = heavy_tailed(d, 2, torch.bfloat16, seed=len(lv), scale=float(lv[-1]) / 8)
        salt_special_values(g, d, p)
        got = tq.tq_compress(g, [p, p], seed=5, first_worker=1, d=d).cpu().numpy().view(np.uint32)
        for i in range(2):
            want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, p), 5, 1 + i)
            assert np.array_equal(got[i], want), lv
    g = heavy_tailed(d, 2, torch.bfloat16, seed=3)
    st = tq.stats_to_host(tq.tq_stats(g, d))
    for mode in (tq.UNIFORM, tq.NONUNIFORM):
        ps = [tq.tq_params(s, 16, mode, 3.0, tq.ALPHA_MAXABS) for s in st]
        got = tq.tq_compress(g, ps, seed=6, d=d).cpu().numpy().view(np.uint32)
        for i in range(2):
            assert np.array_equal(got[i], orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), 6, i))


def test_compress_decision_table_many_workers_mixed_windows(tq, orc):
    """64 workers in one launch whose codebooks need windows of different sizes (scales from 1e-20 to 1e30, centres
    from close to alpha to 40 binades below it): the launch uses the largest window, every row still matches."""
    d, n, L = 262_144 + 33, 64, 8
    rng = np.random.default_rng(7)
    ps, scales = [], []
    for i in range(n):
        a = float(10.0 ** rng.uniform(-20, 30))
        inner = float(10.0 ** rng.uniform(-12, -0.3))
        mags = np.geomspace(a * inner, a, L // 2).astype(F32)
        ps.append(tq.tq_params_from_levels([float(x) for x in np.concatenate([-mags[::-1], mags])]))
        scales.append(a)
    from paper_2402_01798_b200 import inputs
    stride = inputs.worker_stride(d, torch.bfloat16)
    g = torch.zeros((n, stride), dtype=torch.bfloat16, device="cuda")
    for i in range(n):
        inputs.powerlaw_gradient(d, 3.0, scales[i] / 30, 900 + i, "cuda", torch.bfloat16, out=g[i, :d])
    g[:, 11] = float("nan"); g[:, 12] = float("inf"); g[:, 13] = -float("inf"); g[:, 14] = 0.0
    got = tq.tq_compress(g, ps, seed=99, first_worker=0, d=d).cpu().numpy().view(np.uint32)
    for i in range(0, n, 3):
        want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), 99, i)
        assert np.array_equal(got[i], want), (i, scales[i])


@pytest.mark.parametrize("bits,mode", [(2, 0), (3, 1), (4, 1), (4, 0)])
def test_compress_million_elements_and_seed_sensitivity(tq, orc, bits, mode):
    d, n = 1_000_000 + 37, 2
    g = heavy_tailed(d, n, torch.float32, seed=bits)
    _, ps = lib_params_for(tq, g, d, 1 << bits, mode, 3.0)
    a = tq.tq_compress(g, ps, seed=11, d=d).cpu().numpy().view(np.uint32)
    for i in range(n):
        assert np.array_equal(a[i], orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), 11, i))
    b = tq.tq_compress(g, ps, seed=12, d=d).cpu().numpy().view(np.uint32)
    c = tq.tq_compress(g, ps, seed=11, d=d).cpu().numpy().view(np.uint32)
    assert not np.array_equal(a, b) and np.array_equal(a, c)
    # worker index enters the counter: row 1 compressed as "first_worker = 1" equals row 1 of the batch
    single = tq.tq_compress(g[1:2], ps[1:2], seed=11, first_worker=1, d=d).cpu().numpy().view(np.uint32)
    assert np.array_equal(single[0], a[1])


def test_uniform_table_through_nonuniform_kernel(tq, orc):
    """A uniform codebook pushed through the table-search path yields a valid code stream for the same
    quantizer: identical intervals except within rounding of a level (where both answers are the
    paper's quantizer), so the dequantized values differ by less than one ulp-scale amount."""
    d = 200_000
    g = heavy_tailed(d, 1, torch.float32, seed=9)
    _, (pu,) = lib_params_for(tq, g, d, 8, tq.UNIFORM, 3.0)
    pt = tq.tq_params_from_levels([pu.levels[k] for k in range(8)], tq.NONUNIFORM)
    cu = orc.unpack(tq.tq_compress(g, [pu], 3, d=d).cpu().numpy().view(np.uint32)[0], d, 3)
    ct = orc.unpack(tq.tq_compress(g, [pt], 3, d=d).cpu().numpy().view(np.uint32)[0], d, 3)
    assert np.mean(cu != ct) < 1e-4
    want = orc.compress(host_f32(orc, g[0, :d]), to_oracle_params(orc, pt), 3, 0)
    assert np.array_equal(orc.unpack(want, d, 3), ct)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_compress_caller_codebooks_grid_and_search_paths(tq, orc, dtype):
    """Caller-supplied codebooks (Section 3.1's general codebook).  Random ones exercise the lookup
    grid at every resolution; the crowded ones (two levels closer than 1/2048 of the range) force the
    binary-search path; both must give the oracle's codes."""
    rng = np.random.default_rng(2024)
    d = 70_001
    books = []
    for L in (4, 8, 16):
        for trial in range(6):
            a = float(10.0 ** rng.uniform(-4, 0))
            inner = np.sort(rng.uniform(-a, a, L - 2) if trial % 2 else a * np.tanh(rng.normal(0, 10.0 ** rng.uniform(-3, 0), L - 2)))
            lv = np.concatenate([[-a], inner, [a]]).astype(F32)
            if np.all(np.diff(lv) > 0):
                books.append(lv)
        books.append(np.concatenate([[-1.0], np.linspace(0.3, 0.3001, L - 2), [1.0]]).astype(F32))     # crowded
        books.append(np.concatenate([[-2e-3], np.linspace(-1e-7, 1e-7, L - 2), [2e-3]]).astype(F32))  # crowded at 0
    for lv in books:
        p = tq.tq_params_from_levels([float(x) for x in lv])
        g = heavy_tailed(d, 2, dtype, seed=len(lv), scale=float(lv[-1]) / 8)
        salt_special_values(g, d, p)
        got = tq.tq_compress(g, [p, p], seed=77, first_worker=2, d=d).cpu().numpy().view(np.uint32)
        for i in range(2):
            want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, p), 77, 2 + i)
            assert np.array_equal(got[i], want), lv


# ---------------------------------------------------------------------------- decompress-aggregate
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 16, 33, 64])
def test_decompress_aggregate_exact(tq, orc, bits, n):
    L = 1 << bits
    rng = np.random.default_rng(bits * 100 + n)
    # up to 7 tiles of 4096 outputs: direct kernel; from 8 tiles on: bulk-copy kernel (whole tiles, one
    # extra element, ragged tails)
    for d in (1, 7, 8, 31, 32, 33, 255, 257, 4099, 28_672, 28_673, 32_768, 32_769, 65_535, 100_003):
        words = tq.tq_packed_words(d, bits)
        codes = rng.integers(0, L, (n, d), dtype=np.uint8)
        packed_h = np.stack([orc.pack(codes[i], bits) for i in range(n)])
        ps = []
        for i in range(n):
            a = 0.01 * (1 + 0.3 * i)
            mags = np.geomspace(a / 50, a, L // 2).astype(F32) if L > 2 else np.array([a], dtype=F32)
            lv = np.concatenate([-mags[::-1], mags])
            ps.append(tq.tq_params_from_levels([float(x) for x in lv]))
        packed = torch.from_numpy(packed_h.view(np.int32)).cuda()
        out = torch.full((d + 16,), 777.0, dtype=torch.float32, device="cuda")
        tq.tq_decompress_aggregate(packed, d, ps, out=out)
        got = out.cpu().numpy()
        want = orc.decompress_aggregate(packed_h, d, [to_oracle_params(orc, p) for p in ps])
        assert np.all(np.abs(got[:d] - want) <= 1e-6 * np.maximum(np.abs(got[:d]), np.abs(want)))
        assert np.array_equal(got[:d], want)
        assert np.all(got[d:] == 777.0)                    # no write past d
        if n in (3, 8, 33) and d in (33, 4099, 100_003):
            w = rng.random(n).astype(F32); w /= w.sum()
            gw = tq.tq_decompress_aggregate(packed, d, ps, weights=list(w)).cpu().numpy()
            ww = orc.decompress_aggregate(packed_h, d, [to_oracle_params(orc, p) for p in ps], weights=w)
            assert np.array_equal(gw, ww)


@pytest.mark.parametrize("bits,n", [(4, 16), (3, 5), (2, 7), (1, 2)])
def test_decompress_aggregate_rows_in_separate_allocations(tq, orc, bits, n):
    """tq_decompress_aggregate_rows: every worker's row in its own allocation (offset inside it, given in a
    shuffled order of allocation) gives the bytes of the contiguous call and of the oracle."""
    L = 1 << bits
    rng = np.random.default_rng(bits * 7 + n)
    for d in (33, 4099, 100_003):
        words = tq.tq_packed_words(d, bits)
        codes = rng.integers(0, L, (n, d), dtype=np.uint8)
        packed_h = np.stack([orc.pack(codes[i], bits) for i in range(n)])
        ps = []
        for i in range(n):
            a = 0.01 * (1 + 0.3 * i)
            mags = np.geomspace(a / 50, a, L // 2).astype(F32) if L > 2 else np.array([a], dtype=F32)
            ps.append(tq.tq_params_from_levels([float(x) for x in np.concatenate([-mags[::-1], mags])]))
        want = orc.decompress_aggregate(packed_h, d, [to_oracle_params(orc, p) for p in ps])
        bufs = {}
        for i in rng.permutation(n):                                  # allocation order != worker order
            pad = 4 * int(rng.integers(0, 5))                          # 16-byte aligned offset into a larger buffer
            buf = torch.full((pad + words + 8,), -1, dtype=torch.int32, device="cuda")
            buf[pad:pad + words] = torch.from_numpy(packed_h[i].view(np.int32)).cuda()
            bufs[int(i)] = (buf, pad)
        rows = [bufs[i][0][bufs[i][1]:bufs[i][1] + words] for i in range(n)]
        out = torch.full((d + 16,), 777.0, dtype=torch.float32, device="cuda")
        tq.tq_decompress_aggregate_rows(rows, d, ps, out=out)
        got = out.cpu().numpy()
        assert np.array_equal(got[:d], want) and np.all(got[d:] == 777.0)
        ptrs = [r.data_ptr() for r in rows]                            # raw addresses, as a peer mapping would give
        got2 = tq.tq_decompress_aggregate_rows(ptrs, d, ps).cpu().numpy()
        assert np.array_equal(got2, want)
    with pytest.raises(tq.TqError):
        tq.tq_decompress_aggregate_rows([rows[0].data_ptr() + 4] + rows[1:], d, ps)      # misaligned row


# ------------------------------------------------------------------------------- whole round trips
def run_round(tq, g, d, L, mode, gamma, seed):
    st, ps = lib_params_for(tq, g, d, L, mode, gamma)
    packed = tq.tq_compress(g, ps, seed, d=d)
    out = tq.tq_decompress_aggregate(packed, d, ps)
    torch.cuda.synchronize()
    return st, ps, packed, out


def check_params_against_oracle(tq, orc, st, ps, L, mode, gamma):
    for s, p in zip(st, ps):
        o = orc.params(orc.Stats(d=s.d, n_tail=s.n_tail, n_nonfinite=s.n_nonfinite, sum_abs=s.sum_abs, sum_sq=s.sum_sq,
                                 sum_log_tail=s.sum_log_tail, max_abs=s.max_abs, g_min=s.g_min), L, mode, gamma)
        assert o.flags == p.flags and math.isclose(o.alpha, p.alpha, rel_tol=3e-7)
        assert np.allclose(list(o.levels), list(p.levels), rtol=5e-7, atol=0)


def test_config1_small_full(tq, orc):
    """d = 100,000, N = 1, gamma = 3, scale 1e-3, uniform, 4 levels: everything compared in full."""
    from paper_2402_01798_b200 import inputs
    w = inputs.WORKLOADS[0]
    g, _ = inputs.make_worker_gradients(w, "cuda")
    st, ps, packed, out = run_round(tq, g, w.d, w.num_levels, tq.UNIFORM, w.gamma, seed=0)
    x = host_f32(orc, g[0, :w.d])
    o = orc.stats(x)
    assert st[0].n_nonfinite == 0 and st[0].max_abs == o.max_abs
    assert math.isclose(st[0].sum_abs, o.sum_abs, rel_tol=TOL_SUM) and math.isclose(st[0].g_min, o.g_min, rel_tol=TOL_SUM)
    check_params_against_oracle(tq, orc, st, ps, 4, orc.UNIFORM, w.gamma)
    op = to_oracle_params(orc, ps[0])
    want = orc.compress(x, op, 0, 0)
    assert packed.shape == (1, 6252) and np.array_equal(packed.cpu().numpy().view(np.uint32)[0], want)
    agg = orc.decompress_aggregate(want[None, :], w.d, [op])
    assert np.array_equal(out.cpu().numpy(), agg)


@pytest.mark.parametrize("cfg", [1, 2])
def test_config2_config3_full_size(tq, orc, cfg):
    """d = 11.2 M x 8 workers (uniform, 8 levels) and d = 25.6 M x 16 workers (non-uniform, 16 levels) at
    full size, in the launch configuration the benchmark times.  Packed rows are compared in full for
    two workers and on windows for the rest; the aggregate is compared on windows (each output needs
    all N rows)."""
    from paper_2402_01798_b200 import inputs
    w = inputs.WORKLOADS[cfg]
    mode = tq.NONUNIFORM if w.mode == "nonuniform" else tq.UNIFORM
    g, _ = inputs.make_worker_gradients(w, "cuda")
    st, ps, packed, out = run_round(tq, g, w.d, w.num_levels, mode, w.gamma, seed=cfg)
    check_params_against_oracle(tq, orc, st, ps, w.num_levels, mode, w.gamma)
    ops = [to_oracle_params(orc, p) for p in ps]
    bits = ps[0].bits
    for i in (0, w.n_workers - 1):
        want = orc.compress(host_f32(orc, g[i, :w.d]), ops[i], cfg, i)
        assert np.array_equal(packed[i].cpu().numpy().view(np.uint32), want), i
    check_windows(tq, orc, g, w.d, ops, packed, out, seed=cfg, bits=bits, n_windows=6, win=1 << 16)


def check_windows(tq, orc, g, d, ops, packed, out, seed, bits, n_windows, win, first_worker=0):
    """Compare codes and aggregates on 32-aligned windows (start, end, and seeded interior offsets,
    including one that straddles the 2^32-bit offset of the stream when the row is long enough)."""
    n = len(ops)
    rng = np.random.default_rng(seed + 12345)
    starts = [0, max(0, (d - win) // 32 * 32)]
    if d * bits > 2 ** 32 + win * bits:
        starts.append(((2 ** 32 // bits) - win // 2) // 32 * 32)
    if d > 2 ** 31 + win:
        starts.append((2 ** 31 - win // 2) // 32 * 32)
    while len(starts) < n_windows:
        starts.append(int(rng.integers(0, max(1, d - win))) // 32 * 32)
    for a in starts:
        b = min(d, a + win)
        w0, w1 = a * bits // 32, -(-b * bits // 32)
        rows = packed[:, w0:w1].cpu().numpy().view(np.uint32)
        for i in range(n):
            x = host_f32(orc, g[i, a:b])
            want = orc.pack(orc.quantize_window(x, a, ops[i], seed, first_worker + i), bits, words=w1 - w0)
            assert np.array_equal(rows[i], want), (a, i)
        agg = orc.decompress_aggregate(np.ascontiguousarray(rows), b - a, ops)
        got = out[a:b].cpu().numpy()
        assert np.all(np.abs(got - agg) <= 1e-6 * np.maximum(np.abs(got), np.abs(agg)))
        assert np.array_equal(got, agg), a


@pytest.mark.parametrize("gamma,mode,L", [(2.2, "uniform", 4), (3.0, "nonuniform", 16), (4.0, "nonuniform", 4), (2.2, "nonuniform", 16)])
def test_config4_bf16_outliers_windows(tq, orc, gamma, mode, L):
    """d = 124 M bf16 x 8 workers with 1% of entries multiplied by 100: full-size launch, windows compared.
    (gamma = 2.2 with 16 non-uniform levels has no finite fixed point: alpha is capped at max|g|.)"""
    from paper_2402_01798_b200 import inputs
    w = next(c for c in inputs.CONFIG4_SWEEP if c.gamma == gamma and c.mode == mode and c.num_levels == L)
    m = tq.NONUNIFORM if mode == "nonuniform" else tq.UNIFORM
    g, _ = inputs.make_worker_gradients(w, "cuda")
    st, ps, packed, out = run_round(tq, g, w.d, L, m, gamma, seed=44)
    check_params_against_oracle(tq, orc, st, ps, L, m, gamma)
    if gamma == 2.2 and mode == "nonuniform" and L == 16:
        assert all(p.flags & tq.FLAG_ALPHA_CAPPED for p in ps)
    # statistics of one full row against the oracle
    x = host_f32(orc, g[3, :w.d])
    o = orc.stats(x, g_min=st[3].g_min)
    assert st[3].n_tail == o.n_tail and st[3].max_abs == o.max_abs
    assert math.isclose(st[3].sum_abs, o.sum_abs, rel_tol=TOL_SUM) and math.isclose(st[3].sum_log_tail, o.sum_log_tail, rel_tol=TOL_LOG)
    del x
    check_windows(tq, orc, g, w.d, [to_oracle_params(orc, p) for p in ps], packed, out, seed=44, bits=ps[0].bits,
                  n_windows=5, win=1 << 16)


def test_config5_billion_elements_windows(tq, orc):
    """d = 10^9 x 4 workers, non-uniform, 8 levels (3-bit codes crossing word boundaries; element and
    bit offsets beyond 2^32): full-size launch; windows at both ends, across the 2^32-bit offset, and
    at seeded interior offsets."""
    from paper_2402_01798_b200 import inputs
    w = inputs.WORKLOADS[4]
    g, _ = inputs.make_worker_gradients(w, "cuda")
    st, ps, packed, out = run_round(tq, g, w.d, w.num_levels, tq.NONUNIFORM, w.gamma, seed=5)
    check_params_against_oracle(tq, orc, st, ps, 8, tq.NONUNIFORM, w.gamma)
    assert all(s.d == w.d and s.n_nonfinite == 0 for s in st)
    assert packed.shape == (4, 93_750_000)
    check_windows(tq, orc, g, w.d, [to_oracle_params(orc, p) for p in ps], packed, out, seed=5, bits=3,
                  n_windows=7, win=1 << 16)
    # statistics of one full row (10^9 elements) against the oracle
    x = host_f32(orc, g[1, :w.d])
    o = orc.stats(x, g_min=st[1].g_min)
    assert st[1].n_tail == o.n_tail and st[1].max_abs == o.max_abs
    assert math.isclose(st[1].sum_abs, o.sum_abs, rel_tol=TOL_SUM) and math.isclose(st[1].sum_sq, o.sum_sq, rel_tol=TOL_SUM)
    assert math.isclose(st[1].sum_log_tail, o.sum_log_tail, rel_tol=TOL_LOG)


# ----------------------------------------------------------------------- device-resident parameters
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("L,mode,gamma", [(4, 0, 3.0), (8, 0, 2.5), (8, 1, 2.5), (16, 1, 3.0), (16, 1, 2.2), (2, 1, 4.0), (16, 0, float("nan")),
                                          (8, 2, 3.0), (16, 2, 2.5)])
def test_round_without_host_round_trip(tq, orc, dtype, L, mode, gamma):
    """statistics -> tq_params_device -> tq_compress_device_params -> tq_decompress_aggregate_device_params,
    nothing copied to the host in between.  The device-made parameters agree with the host's (and so
    with the oracle's) to fp32 rounding; codes and aggregate are bit-exact against the oracle run on
    the device-made parameters."""
    d, n = 300_007, 5
    g = heavy_tailed(d, n, dtype, seed=L * 7 + mode)
    stats_dev = tq.tq_stats(g, d)
    params_dev = tq.tq_params_device(stats_dev, n, L, mode, gamma)
    packed = tq.tq_compress_device_params(g, params_dev, L, mode, seed=321, first_worker=3, d=d)
    out = tq.tq_decompress_aggregate_device_params(packed, d, params_dev, L)
    torch.cuda.synchronize()
    st = tq.stats_to_host(stats_dev)
    dev_ps = tq.params_to_host(params_dev)
    for s, p in zip(st, dev_ps):
        h = tq.tq_params(s, L, mode, gamma)
        assert p.flags == h.flags and p.bits == h.bits and p.mode == h.mode and p.iterations == h.iterations
        assert math.isclose(p.alpha, h.alpha, rel_tol=3e-7) and math.isclose(p.inv_step, h.inv_step, rel_tol=5e-7)
        assert np.allclose(list(p.levels), list(h.levels), rtol=5e-7, atol=0)
        assert np.allclose(list(p.inv_width), list(h.inv_width), rtol=2e-6, atol=0)
    ops = [to_oracle_params(orc, p) for p in dev_ps]
    got = packed.cpu().numpy().view(np.uint32)
    for i in range(n):
        assert np.array_equal(got[i], orc.compress(host_f32(orc, g[i, :d]), ops[i], 321, 3 + i)), i
    assert np.array_equal(out.cpu().numpy(), orc.decompress_aggregate(got, d, ops))
    # the host-parameter path on the same (device-made) parameters gives the same bytes
    again = tq.tq_compress(g, dev_ps, 321, 3, d=d)
    assert torch.equal(again, packed)
    w = [0.1 * (i + 1) for i in range(n)]
    ow = tq.tq_decompress_aggregate_device_params(packed, d, params_dev, L, weights=w)
    assert torch.equal(ow, tq.tq_decompress_aggregate(packed, d, dev_ps, weights=w))


@pytest.mark.parametrize("L", [4, 8, 16])
def test_biscaled_codebook_through_the_table_kernels(tq, orc, L):
    """Truncated BiScaled quantizer (Appendix): parameters from the library against the oracle's, codes
    and aggregate bit-exact (it is a table codebook to the kernels)."""
    d, n = 400_003, 4
    g = heavy_tailed(d, n, torch.float32, seed=50 + L, gamma=3.5)
    st, ps = lib_params_for(tq, g, d, L, tq.BISCALED, 3.5)
    check_params_against_oracle(tq, orc, st, ps, L, orc.BISCALED, 3.5)
    packed = tq.tq_compress(g, ps, seed=8, d=d)
    out = tq.tq_decompress_aggregate(packed, d, ps)
    ops = [to_oracle_params(orc, p) for p in ps]
    got = packed.cpu().numpy().view(np.uint32)
    for i in range(n):
        assert np.array_equal(got[i], orc.compress(host_f32(orc, g[i, :d]), ops[i], 8, i))
    assert np.array_equal(out.cpu().numpy(), orc.decompress_aggregate(got, d, ops))


@pytest.mark.parametrize("mode", [0, 1])
def test_no_truncation_baselines(tq, orc, mode):
    """alpha = max|g| (QSGD / NQSGD of Section 5) through the same kernels, host and device parameters."""
    d, n = 200_001, 2
    g = heavy_tailed(d, n, torch.float32, seed=31 + mode, gamma=2.5)
    stats_dev = tq.tq_stats(g, d)
    st = tq.stats_to_host(stats_dev)
    ps = [tq.tq_params(s, 8, mode, 2.5, tq.ALPHA_MAXABS) for s in st]
    for s, p in zip(st, ps):
        assert p.alpha == s.max_abs
    got = tq.tq_compress(g, ps, seed=4, d=d).cpu().numpy().view(np.uint32)
    for i in range(n):
        assert np.array_equal(got[i], orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), 4, i))
    pd = tq.tq_params_device(stats_dev, n, 8, mode, 2.5, tq.ALPHA_MAXABS)
    assert [p.alpha for p in tq.params_to_host(pd)] == [p.alpha for p in ps]
    assert torch.equal(tq.tq_compress_device_params(g, pd, 8, mode, seed=4, d=d).cpu(), torch.from_numpy(got.view(np.int32)))


def test_device_params_marks_bad_statistics_and_fallback_codebooks(tq, orc):
    """A worker whose statistics are outside the domain is flagged, its row is all zeros and it adds zero
    to the aggregate; a crowded caller-made codebook written into the device records takes the
    binary-search path inside the device-parameter kernel."""
    d, n = 50_003, 3
    g = heavy_tailed(d, n, torch.float32, seed=77)
    g[1].zero_()                                             # all-zero gradient: g_min = 0, no tail
    stats_dev = tq.tq_stats(g, d)
    params_dev = tq.tq_params_device(stats_dev, n, 8, tq.NONUNIFORM, 3.0)
    ps = tq.params_to_host(params_dev)
    assert ps[1].flags & tq.FLAG_INVALID and ps[1].iterations == tq.ERR_DOMAIN and ps[1].alpha == 0.0
    assert not (ps[0].flags & tq.FLAG_INVALID) and not (ps[2].flags & tq.FLAG_INVALID)
    packed = tq.tq_compress_device_params(g, params_dev, 8, tq.NONUNIFORM, seed=5, d=d)
    out = tq.tq_decompress_aggregate_device_params(packed, d, params_dev, 8)
    got = packed.cpu().numpy().view(np.uint32)
    assert not got[1].any()
    ops = [to_oracle_params(orc, p) for p in ps]
    for i in (0, 2):
        assert np.array_equal(got[i], orc.compress(host_f32(orc, g[i, :d]), ops[i], 5, i))
    acc = np.zeros(d, dtype=F32)
    for i in range(n):
        acc = (acc + np.array(ops[i].levels[:8], dtype=F32)[orc.unpack(got[i], d, 3)]).astype(F32)
    assert np.array_equal(out.cpu().numpy(), (acc / F32(3)).astype(F32))
    # crowded codebook -> binary-search fallback
    lv = np.concatenate([[-1.0], np.linspace(0.3, 0.3001, 6), [1.0]]).astype(F32)
    p = tq.tq_params_from_levels([float(x) for x in lv])
    raw = torch.frombuffer(bytearray(bytes(p) * n), dtype=torch.uint8).cuda()
    g2 = heavy_tailed(d, n, torch.float32, seed=78, scale=0.2)
    pk = tq.tq_compress_device_params(g2, raw, 8, tq.NONUNIFORM, seed=9, d=d).cpu().numpy().view(np.uint32)
    for i in range(n):
        assert np.array_equal(pk[i], orc.compress(host_f32(orc, g2[i, :d]), to_oracle_params(orc, p), 9, i))


@pytest.mark.parametrize("dtype,d", [(torch.float32, 300_007), (torch.bfloat16, 262_144 + 5)])
def test_round_as_cuda_graph_replays_identically(tq, orc, dtype, d):
    """The round without a host round trip (one-pass statistics, device-made parameters, compress, aggregate) captured once
    as a CUDA graph: every replay on new data gives the packed rows and the update of the kernel-by-kernel round."""
    n, L, mode = 4, 16, tq.NONUNIFORM
    g = heavy_tailed(d, n, dtype, seed=5)
    hint = tq.new_gmin_hint(n, "cuda")
    stats_dev = torch.empty(n * 64, dtype=torch.uint8, device="cuda")
    ws = torch.empty(tq.tq_stats_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    params_dev = torch.empty(n * 176, dtype=torch.uint8, device="cuda")
    packed = torch.empty((n, tq.tq_packed_words(d, 4)), dtype=torch.int32, device="cuda")
    out = torch.empty(d, dtype=torch.float32, device="cuda")

    def device_round():
        tq.tq_stats_hinted(g, hint, d, stats_dev=stats_dev, workspace=ws)
        tq.tq_params_device(stats_dev, n, L, mode, 3.0, params_dev=params_dev)
        tq.tq_compress_device_params(g, params_dev, L, mode, seed=77, d=d, packed=packed)
        tq.tq_decompress_aggregate_device_params(packed, d, params_dev, L, out=out)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        device_round()                                   # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        device_round()
    for rnd in range(2):
        g.copy_(heavy_tailed(d, n, dtype, seed=40 + rnd, scale=1e-3 * (1 + rnd)))      # new data, mean in another binade
        graph.replay()
        torch.cuda.synchronize()
        got_packed, got_out = packed.clone(), out.clone()
        ps = tq.params_to_host(params_dev)
        device_round()
        torch.cuda.synchronize()
        assert torch.equal(got_packed, packed) and torch.equal(got_out, out)
        for i in (0, n - 1):
            want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), 77, i)
            assert np.array_equal(got_packed[i].cpu().numpy().view(np.uint32), want)
    assert tq.tq_wait_expired_count() == 0


@pytest.mark.parametrize("L", [4, 16])
def test_device_params_rows_split_between_table_and_element_wise_kernels(tq, orc, L):
    """bf16 rows with device-resident table codebooks: the decision-table kernel serves the rows its window fits and the
    element-wise kernels the others (a codebook whose centre is 100 binades below alpha, a row marked invalid); every row
    matches the oracle and the invalid one is all zeros.  Also through the whole device route from statistics on."""
    d, bits = 262_144 + 77, {4: 2, 16: 4}[L]
    half = L // 2
    books = [np.concatenate([-np.geomspace(0.02, 2e-4, half), np.geomspace(2e-4, 0.02, half)]).astype(F32),
             np.concatenate([-np.geomspace(1.0, 1e-30, half), np.geomspace(1e-30, 1.0, half)]).astype(F32),
             np.concatenate([[-1.0], np.linspace(0.3, 0.3001, L - 2), [1.0]]).astype(F32)]
    ps = [tq.tq_params_from_levels([float(x) for x in lv]) for lv in books]
    bad = tq.Params()
    bad.bits, bad.num_levels, bad.mode, bad.flags = bits, L, tq.NONUNIFORM, 8
    ps.append(bad)
    n = len(ps)
    raw = torch.frombuffer(bytearray(b"".join(bytes(p) for p in ps)), dtype=torch.uint8).cuda()
    g = heavy_tailed(d, n, torch.bfloat16, seed=L, scale=2e-3)
    salt_special_values(g, d, ps[0])
    got = tq.tq_compress_device_params(g, raw, L, tq.NONUNIFORM, seed=21, first_worker=3, d=d).cpu().numpy().view(np.uint32)
    for i in range(n - 1):
        want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, ps[i]), 21, 3 + i)
        assert np.array_equal(got[i], want), i
    assert not got[n - 1].any()
    # statistics -> device parameters -> compress, nothing designed on the host
    g2 = heavy_tailed(d, 3, torch.bfloat16, seed=50 + L)
    pd = tq.tq_params_device(tq.tq_stats(g2, d), 3, L, tq.NONUNIFORM, 3.0)
    got2 = tq.tq_compress_device_params(g2, pd, L, tq.NONUNIFORM, seed=22, d=d).cpu().numpy().view(np.uint32)
    for i, p in enumerate(tq.params_to_host(pd)):
        assert np.array_equal(got2[i], orc.compress(host_f32(orc, g2[i, :d]), to_oracle_params(orc, p), 22, i)), i


@pytest.mark.parametrize("bits,n,mu,wd", [(4, 16, 0.9, 5e-4), (3, 4, 0.9, 0.0), (2, 8, 0.0, 1e-3), (4, 3, 0.0, 0.0), (1, 2, 0.5, 5e-4)])
def test_fused_model_update_matches_oracle(tq, orc, bits, n, mu, wd):
    """tq_decompress_aggregate_apply: aggregation fused with the momentum-SGD step, two rounds in a row,
    theta and the momentum buffer bit-exact against the oracle (ragged d, canaries past the end)."""
    L = 1 << bits
    rng = np.random.default_rng(bits * 31 + n)
    for d in (33, 100_003):
        ps = []
        for i in range(n):
            a = 0.01 * (1 + 0.3 * i)
            mags = np.geomspace(a / 50, a, L // 2).astype(F32) if L > 2 else np.array([a], dtype=F32)
            ps.append(tq.tq_params_from_levels([float(x) for x in np.concatenate([-mags[::-1], mags])]))
        ops = [to_oracle_params(orc, p) for p in ps]
        theta_h = rng.normal(0, 0.1, d).astype(F32)
        buf_h = np.zeros(d, dtype=F32) if mu != 0.0 else None
        theta = torch.full((d + 16,), 5.0, dtype=torch.float32, device="cuda"); theta[:d] = torch.from_numpy(theta_h)
        buf = None
        if mu != 0.0:
            buf = torch.full((d + 16,), -3.0, dtype=torch.float32, device="cuda"); buf[:d] = 0.0
        for rnd in range(2):
            codes = rng.integers(0, L, (n, d), dtype=np.uint8)
            packed_h = np.stack([orc.pack(codes[i], bits) for i in range(n)])
            packed = torch.from_numpy(packed_h.view(np.int32)).cuda()
            tq.tq_decompress_aggregate_apply(packed, d, ps, theta, buf, 0.01, mu, wd)
            orc.decompress_aggregate_apply(packed_h, d, ops, theta_h, buf_h, 0.01, mu, wd)
            assert np.array_equal(theta[:d].cpu().numpy(), theta_h)
            assert bool((theta[d:] == 5.0).all())
            if buf is not None:
                assert np.array_equal(buf[:d].cpu().numpy(), buf_h) and bool((buf[d:] == -3.0).all())


def test_layer_groups_are_quantized_independently(tq, orc):
    """Section 5: convolutional and fully-connected gradients have different distributions and are
    quantized independently.  With row strides in the ABI a layer group is a column range of the
    [N, d] gradient block: one statistics / compress / decompress call per group on a 32-byte aligned
    sub-range, each group with its own alpha and codebook, element indices counted within the group."""
    n, d_conv, d_fc = 4, 60_000, 140_008
    d = d_conv + d_fc
    g = torch.zeros((n, d), dtype=torch.float32, device="cuda")
    from paper_2402_01798_b200 import inputs
    for i in range(n):
        inputs.powerlaw_gradient(d_conv, 4.0, 5e-3, 900 + i, "cuda", out=g[i, :d_conv])       # light tail, large scale
        inputs.powerlaw_gradient(d_fc, 2.5, 2e-4, 950 + i, "cuda", out=g[i, d_conv:])        # heavy tail, small scale
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    alphas = []
    for lo, hi, gamma, L, mode in ((0, d_conv, 4.0, 8, tq.UNIFORM), (d_conv, d, 2.5, 8, tq.NONUNIFORM)):
        view = g[:, lo:hi]
        st = tq.stats_to_host(tq.tq_stats(view))
        ps = [tq.tq_params(s, L, mode, gamma) for s in st]
        alphas.append(ps[0].alpha)
        packed = tq.tq_compress(view, ps, seed=17)
        tq.tq_decompress_aggregate(packed, hi - lo, ps, out=out[lo:hi])
        ops = [to_oracle_params(orc, p) for p in ps]
        got = packed.cpu().numpy().view(np.uint32)
        for i in range(n):
            x = host_f32(orc, g[i, lo:hi])
            o = orc.stats(x, g_min=st[i].g_min)
            assert o.n_tail == st[i].n_tail and math.isclose(o.sum_abs, st[i].sum_abs, rel_tol=TOL_SUM)
            assert np.array_equal(got[i], orc.compress(x, ops[i], 17, i))
        assert np.array_equal(out[lo:hi].cpu().numpy(), orc.decompress_aggregate(got, hi - lo, ops))
    assert max(alphas) > 5 * min(alphas)      # the groups really get different thresholds


def test_no_bounded_wait_ran_out(tq):
    """The bulk-copy decompression kernel gives up on a barrier after a fixed number of polls and counts
    that; in a healthy run (everything above included, when run after it) the count is zero."""
    torch.cuda.synchronize()
    assert tq.tq_wait_expired_count() == 0
