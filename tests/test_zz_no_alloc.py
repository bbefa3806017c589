"""tq_stats_static: the statistics reduction for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside an allocator or
communication callback of a training framework, in a plugin that is given device buffers but may
not create any, or in a step loop where an allocation would stall the device.  For them the library
carries its reduction scratch inside its own device image and offers tq_stats_static, which takes
only the gradient and the output records.

This file is collected last on purpose (its name sorts after the other test files), so a run that
stops at the first failure has already run everything else.  It stands alone: it needs no state
from the other tests and leaves none behind.
"""
import ctypes as C
import math

import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tq():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_01798_b200 import binding
    binding.lib()
    return binding


def _records(tq, dev_bytes):
    return tq.stats_to_host(dev_bytes)


def _same(a, b):
    # both entry points run the same kernels with the same launch shape and fold block records in
    # index order, so the records agree bit for bit; the sums are additionally held to the
    # tolerance the parity tests use for them
    assert (a.d, a.n_tail, a.n_nonfinite) == (b.d, b.n_tail, b.n_nonfinite)
    assert a.max_abs == b.max_abs and a.g_min == b.g_min
    for f, tol in (("sum_abs", 2e-6), ("sum_sq", 2e-6), ("sum_log_tail", 5e-6)):
        assert math.isclose(getattr(a, f), getattr(b, f), rel_tol=tol, abs_tol=1e-12)
        assert getattr(a, f) == getattr(b, f)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_static_scratch_matches_tq_stats_twice_in_a_row(tq, dtype):
    from paper_2402_01798_b200 import inputs
    n, d = 5, 1_000_003
    stride = inputs.worker_stride(d, dtype)
    g = torch.zeros((n, stride), dtype=dtype, device="cuda")
    for i in range(n):
        inputs.powerlaw_gradient(d, 3.0, 1e-3, 4242 + i, "cuda", dtype, out=g[i, :d])
    g[2, 17] = float("nan")
    out_static = torch.empty(n * 64, dtype=torch.uint8, device="cuda")      # the caller's output buffer
    out_ref = torch.empty(n * 64, dtype=torch.uint8, device="cuda")
    ws = torch.empty(tq.tq_stats_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    L = tq.lib()
    stream = torch.cuda.current_stream().cuda_stream
    code = tq.F32 if dtype == torch.float32 else tq.BF16
    for g_min in (0.0, 8e-4):                 # automatic threshold (two passes) and a given one (one pass)
        assert L.tq_stats(g.data_ptr(), code, d, stride, n, g_min, 1.0, out_ref.data_ptr(), ws.data_ptr(), ws.numel(), stream) == tq.OK
        want = _records(tq, out_ref)
        for call in range(2):                 # the second call finds the first call's leftovers in the array
            out_static.fill_(0xEE)
            rc = L.tq_stats_static(g.data_ptr(), code, d, stride, n, g_min, 1.0, out_static.data_ptr(), stream)
            assert rc == tq.OK, L.tq_strerror(rc)
            got = _records(tq, out_static)
            for a, b in zip(got, want):
                _same(a, b)
        # a different, smaller problem in between must not disturb the next call either
        small = torch.empty(64, dtype=torch.uint8, device="cuda")
        assert L.tq_stats_static(g.data_ptr(), code, 4099, stride, 1, g_min, 1.0, small.data_ptr(), stream) == tq.OK
        rc = L.tq_stats_static(g.data_ptr(), code, d, stride, n, g_min, 1.0, out_static.data_ptr(), stream)
        assert rc == tq.OK
        for a, b in zip(_records(tq, out_static), want):
            _same(a, b)


def test_static_scratch_limit_is_reported(tq):
    L = tq.lib()
    n = tq.STATIC_MAX_WORKERS + 1
    g = torch.zeros((n, 64), dtype=torch.float32, device="cuda")
    out = torch.full((n * 64,), 0x11, dtype=torch.uint8, device="cuda")
    rc = L.tq_stats_static(g.data_ptr(), tq.F32, 64, 64, n, 0.0, 1.0, out.data_ptr(), None)
    assert rc == tq.ERR_STATIC_LIMIT
    assert b"16" in L.tq_strerror(rc)
    torch.cuda.synchronize()
    assert bool((out == 0x11).all())          # nothing was launched
    # exactly the maximum is fine
    g16 = torch.rand((tq.STATIC_MAX_WORKERS, 4096), device="cuda") - 0.5
    out16 = torch.empty(tq.STATIC_MAX_WORKERS * 64, dtype=torch.uint8, device="cuda")
    tq.tq_stats_static(g16, out16)
    ref = tq.stats_to_host(tq.tq_stats(g16))
    for a, b in zip(tq.stats_to_host(out16), ref):
        _same(a, b)
