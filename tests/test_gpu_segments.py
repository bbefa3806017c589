"""GPU parity of the layer-group calls (Section 5: groups of layers are quantized independently): statistics,
parameters, compression and aggregation of every (worker, segment) pair in one launch per step, against the
CPU oracle run on each segment by itself and against the library's own one-call-per-group route."""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

F32 = np.float32
TOL_SUM, TOL_LOG = 2e-6, 5e-6


@pytest.fixture(scope="module")
def tq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_01798_b200 import binding
    binding.lib()
    return binding


def to_oracle_params(orc, p):
    q = orc.Params()
    for f in ("bits", "num_levels", "mode", "flags", "alpha", "inv_step", "gamma", "g_min", "rho", "iterations"):
        setattr(q, f, getattr(p, f))
    for k in range(16):
        q.levels[k] = p.levels[k]
        q.inv_width[k] = p.inv_width[k]
    return q


def host_f32(orc, t):
    if t.dtype == torch.bfloat16:
        return orc.bf16_to_f32(t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))
    return t.cpu().numpy()


def make_rows(n, width, dtype, seed):
    """Rows whose scale changes along the row, so that the groups really have different distributions."""
    from paper_2402_01798_b200 import inputs
    g = torch.zeros((n, width), dtype=dtype, device="cuda")
    for i in range(n):
        inputs.powerlaw_gradient(width, 3.0, 1e-3, seed + i, "cuda", dtype, out=g[i])
    ramp = torch.logspace(-1.5, 1.0, width, device="cuda")
    return (g.float() * ramp).to(dtype)


TWO_GROUPS = [(0, 120_000), (120_000, 79_991)]
SIXTEEN = [(0, 1), (16, 31), (64, 33), (128, 4096), (4224, 8191), (12416, 8193), (20624, 100), (20736, 50_001),
           (70752, 7), (70768, 32), (70800, 32_768), (103568, 65_537), (169120, 3), (169136, 1000), (170144, 20_000),
           (190144, 9_849)]
OUT_OF_ORDER_WITH_GAPS = [(100_000, 50_003), (0, 30_000), (40_000, 17)]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("L,mode", [(16, 1), (8, 0), (4, 1), (2, 0)])
@pytest.mark.parametrize("table", [TWO_GROUPS, SIXTEEN, OUT_OF_ORDER_WITH_GAPS], ids=["two", "sixteen", "gaps"])
def test_segments_match_oracle_and_per_group_calls(tq, orc, dtype, L, mode, table):
    n, width, bits = 3, 200_000, {2: 1, 4: 2, 8: 3, 16: 4}[L]
    g = make_rows(n, width, dtype, seed=L + len(table))
    S = len(table)
    seed, first = 0xABCDEF12345, 4

    # statistics: one record per (worker, segment)
    st = tq.stats_to_host(tq.tq_stats_segments(g, table))
    assert len(st) == n * S
    for i in range(n):
        for s, (off, ln) in enumerate(table):
            r = st[i * S + s]
            o = orc.stats(host_f32(orc, g[i, off:off + ln]))
            assert r.d == ln and r.n_nonfinite == 0 and r.max_abs == o.max_abs
            assert math.isclose(r.sum_abs, o.sum_abs, rel_tol=TOL_SUM) and math.isclose(r.sum_sq, o.sum_sq, rel_tol=2 * TOL_SUM)
            if r.g_min == o.g_min:          # the mean, hence g_min, may differ in the last bit
                assert r.n_tail == o.n_tail and math.isclose(r.sum_log_tail, o.sum_log_tail, rel_tol=TOL_LOG, abs_tol=1e-9)
            one = tq.stats_to_host(tq.tq_stats(g[i:i + 1, off:off + ln], ln))[0]      # the per-group call on the sub-range
            assert (one.d, one.n_tail, one.max_abs, one.g_min) == (r.d, r.n_tail, r.max_abs, r.g_min)
            assert math.isclose(one.sum_abs, r.sum_abs, rel_tol=1e-12) and math.isclose(one.sum_log_tail, r.sum_log_tail, rel_tol=1e-9, abs_tol=1e-12)

    # parameters on the device, one thread per pair
    stats_dev = tq.tq_stats_segments(g, table)
    params_dev = tq.tq_params_device(stats_dev, n * S, L, mode, 3.0)
    ps = tq.params_to_host(params_dev)
    valid = [not (p.flags & 8) for p in ps]
    assert sum(valid) >= n * (S - 6)                     # only the tiny groups may be outside the model's domain
    for i in range(n):
        for s, (off, ln) in enumerate(table):
            if valid[i * S + s]:
                o = orc.params(orc.stats(host_f32(orc, g[i, off:off + ln]), g_min=st[i * S + s].g_min), L, mode, 3.0)
                assert math.isclose(ps[i * S + s].alpha, o.alpha, rel_tol=2e-6)

    # compression: every pair's packed segment against the oracle and against the per-group call
    total = tq.tq_segments_packed_words(table, bits)
    packed = torch.full((n, total + 8), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    tq.tq_compress_segments(g, table, params_dev, L, mode, seed, first, packed=packed)
    got = packed.cpu().numpy().view(np.uint32)
    assert np.all(got[:, total:] == 0x5A5A5A5A)
    woff = np.concatenate([[0], np.cumsum([tq.tq_packed_words(ln, bits) for _, ln in table])]).astype(int)
    for i in range(n):
        for s, (off, ln) in enumerate(table):
            mine = got[i, woff[s]:woff[s + 1]]
            if not valid[i * S + s]:
                assert not mine.any()
                continue
            want = orc.compress(host_f32(orc, g[i, off:off + ln]), to_oracle_params(orc, ps[i * S + s]), seed, first + i)
            assert np.array_equal(mine, want), (i, s)
    for s, (off, ln) in enumerate(table):                # the same bytes as one call per group
        sub = torch.stack([params_dev.view(n * S, -1)[i * S + s] for i in range(n)]).contiguous().view(-1)
        per_group = tq.tq_compress_device_params(g[:, off:off + ln], sub, L, mode, seed, first, d=ln).cpu().numpy().view(np.uint32)
        assert np.array_equal(per_group, got[:, woff[s]:woff[s + 1]]), s

    # aggregation: every segment's slice of the output; elements between segments are left alone
    out = torch.full((width + 8,), 123.0, dtype=torch.float32, device="cuda")
    tq.tq_decompress_aggregate_segments(packed, table, params_dev, L, out=out)
    res = out.cpu().numpy()
    covered = np.zeros(width + 8, dtype=bool)
    for s, (off, ln) in enumerate(table):
        rows = np.ascontiguousarray(got[:, woff[s]:woff[s + 1]])
        want = orc.decompress_aggregate(rows, ln, [to_oracle_params(orc, ps[i * S + s]) for i in range(n)])
        assert np.array_equal(res[off:off + ln], want), s
        covered[off:off + ln] = True
    assert np.all(res[~covered] == 123.0)
    torch.cuda.synchronize()
    assert tq.tq_wait_expired_count() == 0


def test_segments_with_weights_and_many_pairs(tq, orc):
    """64 segments x 5 workers (320 pairs: more than one launch's worth of by-value quantizers), weighted aggregation."""
    n, L, bits, mode = 5, 16, 4, 1
    ln = 3_008
    table = [(s * 3_072, ln + (s % 7)) for s in range(64)]
    width = 64 * 3_072
    g = make_rows(n, width, torch.float32, seed=99)
    S = len(table)
    stats_dev = tq.tq_stats_segments(g, table)
    params_dev = tq.tq_params_device(stats_dev, n * S, L, mode, 3.0)
    ps = tq.params_to_host(params_dev)
    assert not any(p.flags & 8 for p in ps)
    packed = tq.tq_compress_segments(g, table, params_dev, L, mode, seed=3)
    got = packed.cpu().numpy().view(np.uint32)
    woff = np.concatenate([[0], np.cumsum([tq.tq_packed_words(x, bits) for _, x in table])]).astype(int)
    w = [0.1, 0.3, 0.2, 0.25, 0.15]
    out = torch.zeros(width, dtype=torch.float32, device="cuda")
    tq.tq_decompress_aggregate_segments(packed, table, params_dev, L, out=out, weights=w)
    res = out.cpu().numpy()
    for s, (off, x) in enumerate(table):
        for i in (0, n - 1):
            want = orc.compress(host_f32(orc, g[i, off:off + x]), to_oracle_params(orc, ps[i * S + s]), 3, i)
            assert np.array_equal(got[i, woff[s]:woff[s + 1]], want)
        agg = orc.decompress_aggregate(np.ascontiguousarray(got[:, woff[s]:woff[s + 1]]), x,
                                       [to_oracle_params(orc, ps[i * S + s]) for i in range(n)], weights=w)
        assert np.array_equal(res[off:off + x], agg)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("table", [TWO_GROUPS, SIXTEEN], ids=["two", "sixteen"])
def test_one_pass_statistics_per_segment(tq, orc, dtype, table):
    """tq_stats_hinted_segments: per (worker, segment) the record of the oracle under the power-of-two threshold rule,
    whether the hint is missing, fresh or stale (the record does not depend on it, bit for bit)."""
    n, width = 3, 200_000
    g = make_rows(n, width, dtype, seed=17)
    S = len(table)
    hint = tq.new_gmin_hint(n * S, "cuda")
    first = tq.stats_to_host(tq.tq_stats_hinted_segments(g, table, hint))           # no hint: every pair takes the tail pass
    again = tq.stats_to_host(tq.tq_stats_hinted_segments(g, table, hint))           # hint from the same data: one pass
    hits = [hit for _, hit in tq.gmin_hint_to_host(hint)]
    for i in range(n):
        for s, (off, ln) in enumerate(table):
            a, b = first[i * S + s], again[i * S + s]
            assert bytes(a) == bytes(b), (i, s)
            o = orc.stats_pow2(host_f32(orc, g[i, off:off + ln]))
            assert a.d == ln and a.g_min == o.g_min and a.n_tail == o.n_tail and a.max_abs == o.max_abs
            assert math.isclose(a.sum_abs, o.sum_abs, rel_tol=TOL_SUM)
            assert math.isclose(a.sum_log_tail, o.sum_log_tail, rel_tol=TOL_LOG, abs_tol=1e-9)
            if a.g_min > 0:
                assert hits[i * S + s] == 1
    g2 = (g.float() * 37.0).to(dtype)                                                # the mean moves five binades: stale hints
    stale = tq.stats_to_host(tq.tq_stats_hinted_segments(g2, table, hint))
    fresh = tq.stats_to_host(tq.tq_stats_hinted_segments(g2, table, tq.new_gmin_hint(n * S, "cuda")))
    assert all(bytes(x) == bytes(y) for x, y in zip(stale, fresh))


def test_segment_argument_checks(tq):
    g = torch.zeros((2, 4096), dtype=torch.float32, device="cuda")
    for bad, status in (([(0, 0)], tq.ERR_INVALID_ARG), ([(4, 100)], tq.ERR_ALIGNMENT), ([(0, 100), (96, 50)], tq.ERR_INVALID_ARG),
                        ([(4000, 200)], tq.ERR_INVALID_ARG), ([(8 * k, 8) for k in range(65)], tq.ERR_INVALID_ARG)):
        with pytest.raises(tq.TqError) as e:
            tq.tq_stats_segments(g, bad)
        assert e.value.status == status, bad
    gb = torch.zeros((2, 4096), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tq.TqError) as e:
        tq.tq_stats_segments(gb, [(8, 64)])              # 16 bytes into a bf16 row
    assert e.value.status == tq.ERR_ALIGNMENT
