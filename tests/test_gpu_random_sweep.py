"""Seeded random sweep of the whole path against the oracle: sizes from 1 to 400 000 elements (direct and
bulk / tiled-copy kernels, ragged tails), 1 to 33 workers, 1 to 4 bits, both modes, fp32 and bf16 storage,
NaN / Inf / zero salted in, statistics by either entry point.  Codes and aggregates bit-exact; the
row-pointer aggregation and the device-parameter round must agree with them."""
import numpy as np
import pytest
import torch

from test_gpu_parity import host_f32, to_oracle_params, tq  # noqa: F401  (tq is the library fixture)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("chunk", range(4))
def test_random_configurations(tq, orc, chunk):
    from paper_2402_01798_b200 import inputs
    rng = np.random.default_rng(20240 + chunk)
    done = 0
    for case in range(30):
        bits = int(rng.integers(1, 5)); L = 1 << bits
        mode = int(rng.integers(0, 2))
        dtype = [torch.float32, torch.bfloat16][int(rng.integers(0, 2))]
        n = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 16, 17, 33]))
        d = int(rng.choice([rng.integers(1, 5000), rng.integers(5000, 70_000), rng.integers(60_000, 400_000)]))
        if n * d > 4_000_000:
            n = max(1, 4_000_000 // d)
        g = torch.zeros((n, inputs.worker_stride(d, dtype)), dtype=dtype, device="cuda")
        for i in range(n):
            inputs.powerlaw_gradient(d, float(rng.choice([2.2, 2.5, 3.0, 4.0])), float(rng.choice([1e-4, 1e-3, 1.0])),
                                     100_000 * chunk + 1000 * case + i, "cuda", dtype, out=g[i, :d])
        if d > 8:
            idx = rng.integers(0, d, 3)
            g[:, int(idx[0])] = float("nan"); g[:, int(idx[1])] = float("inf"); g[0, int(idx[2])] = 0.0
        hinted = bool(rng.integers(0, 2))
        if hinted:
            hint = tq.new_gmin_hint(n)
            tq.tq_stats_hinted(g, hint, d)
            sd = tq.tq_stats_hinted(g, hint, d)
        else:
            sd = tq.tq_stats(g, d)
        st = tq.stats_to_host(sd)
        try:
            ps = [tq.tq_params(s, L, mode, float("nan") if rng.integers(0, 2) else 3.0) for s in st]
        except tq.TqError:
            continue                                  # e.g. a single element: no tail to fit
        seed = 7919 * case + chunk
        packed = tq.tq_compress(g, ps, seed=seed, first_worker=2, d=d)
        out = tq.tq_decompress_aggregate(packed, d, ps)
        ph = packed.cpu().numpy().view(np.uint32)
        ops = [to_oracle_params(orc, p) for p in ps]
        for i in range(n):
            x = host_f32(orc, g[i, :d])
            so = orc.stats_pow2(x) if hinted else orc.stats(x)
            assert so.n_nonfinite == st[i].n_nonfinite
            if st[i].g_min == so.g_min:
                assert so.n_tail == st[i].n_tail
            want = orc.compress(x, ops[i], seed, 2 + i)
            assert np.array_equal(ph[i, :want.size], want), (case, i, bits, mode, dtype, d, n)
        agg = orc.decompress_aggregate(ph, d, ops)
        assert np.array_equal(out.cpu().numpy(), agg), (case, bits, mode, dtype, d, n)
        rows = [packed[i].clone() for i in range(n)]
        assert np.array_equal(tq.tq_decompress_aggregate_rows(rows, d, ps).cpu().numpy(), agg)
        pdev = tq.tq_params_device(sd, n, L, mode, 3.0)
        pd = tq.params_to_host(pdev)
        if all(not (p.flags & tq.FLAG_INVALID) for p in pd):
            ph2 = tq.tq_compress_device_params(g, pdev, L, mode, seed=5, first_worker=1, d=d).cpu().numpy().view(np.uint32)
            for i in range(n):
                want = orc.compress(host_f32(orc, g[i, :d]), to_oracle_params(orc, pd[i]), 5, 1 + i)
                assert np.array_equal(ph2[i, :want.size], want), ("device params", case, i)
        done += 1
    assert done >= 20
    torch.cuda.synchronize()
    assert tq.tq_wait_expired_count() == 0
