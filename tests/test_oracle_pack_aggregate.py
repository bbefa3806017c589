"""Pins for the oracle's wire format and server-side aggregation (Algorithm 1, server step).

The wire format is checked against its plain definition written as a Python big integer
(bit i of the stream is bit i of one huge number), the aggregation against NumPy's own fp32
scalars added one worker at a time and against a float64 mean.
"""
import itertools

import numpy as np
import pytest

F32 = np.float32


def _stream_int(codes, bits):
    big = 0
    for j, c in enumerate(codes):
        big |= int(c) << (j * bits)
    return big


def _words_int(words):
    return sum(int(w) << (32 * i) for i, w in enumerate(words))


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("d", [0, 1, 3, 10, 11, 21, 31, 32, 33, 127, 128, 1000, 100_003])
def test_pack_is_lsb_first_dense_stream(orc, bits, d):
    rng = np.random.default_rng(d * 7 + bits)
    codes = rng.integers(0, 1 << bits, d, dtype=np.uint8)
    words = orc.pack(codes, bits)
    assert words.size == orc.packed_words(d, bits) == (-(-d * bits // 32) + 3) // 4 * 4
    assert _words_int(words) == _stream_int(codes, bits)          # also proves the padding is zero
    assert np.array_equal(orc.unpack(words, d, bits), codes)


def test_pack_exhaustive_small(orc):
    """Every code vector for b = 2, d = 8 and b = 3, d = 5; and every 3-bit code at the two
    positions that straddle a 32-bit word boundary (bit offsets 30 and 63)."""
    for bits, d in ((2, 8), (3, 5)):
        for codes in itertools.product(range(1 << bits), repeat=d):
            words = orc.pack(np.array(codes, dtype=np.uint8), bits)
            assert _words_int(words) == _stream_int(codes, bits)
    base = np.zeros(32, dtype=np.uint8)
    for j in (10, 21):                                               # bits 30..32 and 63..65
        assert (j * 3) // 32 != (j * 3 + 2) // 32
        for c in range(8):
            codes = base.copy()
            codes[j] = c
            words = orc.pack(codes, 3)
            assert _words_int(words) == c << (3 * j)
            assert np.array_equal(orc.unpack(words, 32, 3), codes)


def test_compress_is_quantize_then_pack(orc):
    rng = np.random.default_rng(0)
    m = orc.Model(1e-3, 0.1, 3.0)
    for L, mode, d in ((4, orc.UNIFORM, 1000), (8, orc.NONUNIFORM, 4099), (16, orc.NONUNIFORM, 33)):
        p = orc.build_table(m, L, mode, 0.01)
        g = (rng.standard_t(3.0, d) * 1e-3).astype(F32)
        words = orc.compress(g, p, seed=5, worker=1)
        assert _words_int(words) == _stream_int(orc.quantize(g, p, 5, 1), p.bits)
        assert not np.array_equal(words, orc.compress(g, p, seed=5, worker=2))
        assert not np.array_equal(words, orc.compress(g, p, seed=6, worker=1))
        assert np.array_equal(words, orc.compress(g, p, seed=5, worker=1))   # reproducible


def _tables(orc, n, L, mode):
    m = orc.Model(1e-3, 0.1, 3.0)
    return [orc.build_table(m, L, mode, 0.004 * (1 + 0.37 * i)) for i in range(n)]


def test_single_worker_aggregate_is_table_lookup(orc):
    rng = np.random.default_rng(1)
    for L in (4, 8, 16):
        (p,) = _tables(orc, 1, L, orc.NONUNIFORM)
        codes = rng.integers(0, L, 777, dtype=np.uint8)
        out = orc.decompress_aggregate(orc.pack(codes, p.bits)[None, :], 777, [p])
        assert np.array_equal(out, p.levels_np()[codes])             # (0 + v) / 1 is exact


@pytest.mark.parametrize("n", [2, 3, 8, 16])
@pytest.mark.parametrize("bits", [2, 3, 4])
def test_aggregate_is_worker_order_fp32_sum_over_n(orc, n, bits):
    """out_j = (sum_i l^{(i)}[c_ij]) / N with w_i = 1/N (Lemma 2): fp32 adds in worker order, one
    division; also within 1e-6 of the float64 mean."""
    rng = np.random.default_rng(n * 10 + bits)
    L, d = 1 << bits, 501
    ps = _tables(orc, n, L, orc.NONUNIFORM if bits > 2 else orc.UNIFORM)
    codes = rng.integers(0, L, (n, d), dtype=np.uint8)
    packed = np.stack([orc.pack(codes[i], bits) for i in range(n)])
    out = orc.decompress_aggregate(packed, d, ps)
    lv = np.stack([p.levels_np() for p in ps])
    acc = np.zeros(d, dtype=F32)
    for i in range(n):
        acc = (acc + lv[i][codes[i]]).astype(F32)
    assert np.array_equal(out, (acc / F32(n)).astype(F32))
    exact = np.mean([lv[i].astype(np.float64)[codes[i]] for i in range(n)], axis=0)
    scale = max(p.alpha for p in ps)
    assert np.all(np.abs(out - exact) <= 1e-6 * np.abs(exact) + 2e-7 * scale)


def test_aggregate_order_matters_and_is_worker_order(orc):
    """Three values whose fp32 sum depends on the order: (big + -big) + tiny != big + (-big + tiny)."""
    big, tiny = F32(1.0), F32(3e-8)
    ps = [orc.table_params([-big, big]), orc.table_params([-big, big]), orc.table_params([-tiny, tiny])]
    d = 4
    codes = [np.ones(d, np.uint8), np.zeros(d, np.uint8), np.ones(d, np.uint8)]   # +1, -1, +tiny
    packed = np.stack([orc.pack(c, 1) for c in codes])
    out = orc.decompress_aggregate(packed, d, ps)
    assert np.all(out == F32(tiny) / F32(3))
    out2 = orc.decompress_aggregate(packed[[0, 2, 1]], d, [ps[0], ps[2], ps[1]])   # +1, +tiny, -1
    assert np.all(out2 == F32(0.0))                                  # 1 + 3e-8 rounds to 1 in fp32


def test_weighted_aggregate(orc):
    """General weights w_i of the problem statement: sum_i w_i * v_i, products rounded to fp32."""
    rng = np.random.default_rng(3)
    n, d, bits = 5, 300, 3
    ps = _tables(orc, n, 8, orc.NONUNIFORM)
    w = rng.random(n).astype(F32)
    w /= w.sum()
    codes = rng.integers(0, 8, (n, d), dtype=np.uint8)
    packed = np.stack([orc.pack(codes[i], bits) for i in range(n)])
    out = orc.decompress_aggregate(packed, d, ps, weights=w)
    acc = np.zeros(d, dtype=F32)
    for i in range(n):
        acc = (acc + (w[i] * ps[i].levels_np()[codes[i]]).astype(F32)).astype(F32)
    assert np.array_equal(out, acc)


def test_round_trip_mean_is_close_to_clipped_mean(orc):
    """End to end on the oracle alone: many workers compressing the same vector average back to the
    truncated vector (unbiasedness through pack / unpack / aggregate)."""
    rng = np.random.default_rng(4)
    d, n = 2000, 64
    g = (rng.standard_t(3.0, d) * 1e-3).astype(F32)
    st = orc.stats(g)
    p = orc.params(st, 8, orc.NONUNIFORM, gamma=4.0)
    packed = np.stack([orc.compress(g, p, seed=9, worker=i) for i in range(n)])
    out = orc.decompress_aggregate(packed, d, [p] * n)
    clip = np.clip(g, -p.alpha, p.alpha)
    widths = np.diff(p.levels_np()).max()
    assert np.abs(out - clip).max() < 5 * widths / 2 / np.sqrt(n)
    assert abs(np.mean(out - clip)) < 4 * widths / 2 / np.sqrt(n * d)


def _sgd_reference(theta, buf, g, lr, mu, wd):
    """fp32 momentum SGD with weight decay, one NumPy fp32 operation per step (independent restatement)."""
    g = g.astype(F32)
    if wd != 0.0:
        g = (g + (F32(wd) * theta).astype(F32)).astype(F32)
    if buf is not None:
        buf[:] = ((F32(mu) * buf).astype(F32) + g).astype(F32)
        g = buf
    theta[:] = (theta - (F32(lr) * g).astype(F32)).astype(F32)


@pytest.mark.parametrize("mu,wd", [(0.9, 5e-4), (0.0, 0.0), (0.9, 0.0), (0.0, 1e-2)])
def test_fused_model_update_is_momentum_sgd(orc, mu, wd):
    """Algorithm 1's last step with the optimiser of Section 5 (momentum SGD, lr 0.01, momentum 0.9,
    weight decay 5e-4): three rounds in a row against a step-by-step fp32 restatement and against
    torch.optim.SGD (which may fuse a multiply-add: compared to 1e-6)."""
    import torch
    rng = np.random.default_rng(5)
    n, d, bits = 4, 1237, 3
    ps = _tables(orc, n, 8, orc.NONUNIFORM)
    theta = rng.normal(0, 0.1, d).astype(F32)
    use_buf = mu != 0.0
    buf = np.zeros(d, dtype=F32) if use_buf else None
    th_ref, buf_ref = theta.copy(), (buf.copy() if use_buf else None)
    pt = torch.nn.Parameter(torch.from_numpy(theta.copy()))
    opt = torch.optim.SGD([pt], lr=0.01, momentum=mu, weight_decay=wd)
    for rnd in range(3):
        codes = rng.integers(0, 8, (n, d), dtype=np.uint8)
        packed = np.stack([orc.pack(codes[i], bits) for i in range(n)])
        gbar = orc.decompress_aggregate(packed, d, ps)
        orc.decompress_aggregate_apply(packed, d, ps, theta, buf, 0.01, mu, wd)
        _sgd_reference(th_ref, buf_ref, gbar, 0.01, mu, wd)
        assert np.array_equal(theta, th_ref)
        if use_buf:
            assert np.array_equal(buf, buf_ref)
        pt.grad = torch.from_numpy(gbar.copy())
        opt.step()
        assert np.allclose(theta, pt.detach().numpy(), rtol=1e-6, atol=1e-9)


def test_oracle_outputs_match_the_stored_checksums():
    """tests/golden/oracle_small_case.txt is written by tests/golden/make_oracle_golden.py from the oracle
    alone; a mismatch means the oracle's arithmetic (or its inputs) changed."""
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(__file__), "golden")
    spec = importlib.util.spec_from_file_location("make_oracle_golden", os.path.join(here, "make_oracle_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = open(os.path.join(here, "oracle_small_case.txt")).read().splitlines()
    assert mod.lines() == stored
