"""Pins for the oracle's load step and its windowed quantizer entry.

``orc_bf16_to_f32`` is the oracle's first step for gradients stored as bf16 (the 16 stored bits are the
high half of the fp32 pattern); ``orc_quantize_window`` quantizes a window of a longer vector with the
random draw of Section 3.1's quantizer taken per ABSOLUTE element index.  Neither is compared with
itself here: the conversion is checked against integer arithmetic in NumPy and against PyTorch's own
bfloat16 -> float32 conversion for every one of the 65 536 bit patterns, and the window against the
whole-vector quantizer, against the per-element entry, and against a code rebuilt from the Philox block
of the absolute index (the generator itself is pinned in test_oracle_philox.py).
"""
import numpy as np
import pytest
import torch


def test_bf16_to_f32_all_bit_patterns(orc):
    """Every bf16 pattern b becomes the fp32 pattern b << 16, NaN payloads and signed zeros included."""
    raw = np.arange(1 << 16, dtype=np.uint16)
    got = orc.bf16_to_f32(raw).view(np.uint32)
    want_int = raw.astype(np.uint32) << np.uint32(16)                   # integer arithmetic only
    assert np.array_equal(got, want_int)
    # PyTorch's own widening of the same 16-bit patterns, compared as raw bits (NaN != NaN as floats)
    t = torch.from_numpy(raw.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32)
    want_torch = t.view(torch.int32).numpy().view(np.uint32)
    assert np.array_equal(got, want_torch)
    # what widening must keep: the value.  Finite patterns round back to the same bf16 pattern.
    finite = np.isfinite(orc.bf16_to_f32(raw))
    back = torch.from_numpy(orc.bf16_to_f32(raw)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(back[finite], raw[finite])
    assert finite.sum() == 2 * (0x7F80)                                  # all but the two Inf and the NaN patterns


def test_bf16_to_f32_order_and_length(orc):
    """Element i of the output comes from element i of the input (no swap of neighbours), any length."""
    rng = np.random.default_rng(5)
    for n in (0, 1, 2, 3, 7, 8, 9, 1001):
        raw = rng.integers(0, 1 << 16, n, dtype=np.uint16)
        out = orc.bf16_to_f32(raw).view(np.uint32)
        assert out.shape == (n,)
        for i in range(n):
            assert int(out[i]) == int(raw[i]) << 16


def _tables(orc):
    m = orc.Model(1e-3, 0.12, 3.0)
    return [orc.build_table(m, 4, orc.UNIFORM, 0.004), orc.build_table(m, 8, orc.NONUNIFORM, 0.02),
            orc.build_table(m, 16, orc.NONUNIFORM, 0.03), orc.build_table(m, 16, orc.UNIFORM, 0.01)]


def _gradient(rng, n, alpha):
    g = rng.standard_t(2.5, n).astype(np.float32) * np.float32(alpha / 4)
    g[::97] = np.float32(alpha)
    g[1::89] = np.float32(-3 * alpha)
    return g


@pytest.mark.parametrize("a,b", [(0, 41), (3, 77), (5, 1000), (13, 21), (64, 65), (999, 1000), (0, 1000), (7, 7)])
def test_window_equals_slice_of_whole_vector(orc, a, b):
    """quantize_window(g[a:b], a) == quantize(g)[a:b]: windows starting off a multiple of 8 (inside a
    Philox block), at 0, ending at d, of one element, and empty."""
    rng = np.random.default_rng(11)
    for p in _tables(orc):
        g = _gradient(rng, 1000, p.alpha)
        for worker, seed in ((0, 0), (3, 0xDEADBEEF12345678)):
            whole = orc.quantize(g, p, seed, worker)
            win = orc.quantize_window(g[a:b], a, p, seed, worker)
            assert win.dtype == np.uint8 and win.shape == (b - a,)
            assert np.array_equal(win, whole[a:b])


def test_window_differs_when_shifted_by_one(orc):
    """The pin above has teeth: the same values placed one index later draw other random bits."""
    rng = np.random.default_rng(12)
    p = _tables(orc)[2]
    g = rng.uniform(-p.alpha, p.alpha, 4000).astype(np.float32)
    a = orc.quantize_window(g, 40, p, 9, 1)
    b = orc.quantize_window(g, 41, p, 9, 1)
    assert np.count_nonzero(a != b) > 400          # about half of the elements round the other way


@pytest.mark.parametrize("j0", [(1 << 32) + 5, (1 << 35) + 3, (1 << 36) - 2, (1 << 40) - 50])
def test_window_beyond_32_bit_indices(orc, j0):
    """Windows that start beyond 2^32 (and beyond 2^35, where the Philox block index needs its second
    counter word): element by element equal to the per-element entry, and to a code rebuilt here from the
    Philox block of the ABSOLUTE index (counter = (block low, block high, worker, 0), slot = index & 7)
    and the per-value decision."""
    rng = np.random.default_rng(13)
    seed, worker = 0x0123456789ABCDEF, 2
    key = (seed & 0xFFFFFFFF, seed >> 32)
    for p in _tables(orc):
        g = _gradient(rng, 45, p.alpha)
        win = orc.quantize_window(g, j0, p, seed, worker)
        for i in range(g.size):
            j = j0 + i
            assert int(win[i]) == orc.code_at(p, float(g[i]), seed, worker, j)
            block = j >> 3
            out = orc.philox4x32_10((block & 0xFFFFFFFF, block >> 32, worker, 0), key)
            word = int(out[(j & 7) >> 1])
            r16 = (word >> 16) if (j & 1) else (word & 0xFFFF)
            _, k, _, T = orc.decision(p, float(g[i]))
            assert int(win[i]) == k + (1 if r16 < T else 0)
