"""The path with its N workers spread over ranks, on CPU: two and three gloo ranks.

Each rank quantizes and packs only the workers it owns (with the oracle standing in for the kernels:
there is no GPU here), the packed rows and parameter records are all-gathered by
paper_2402_01798_b200.exchange, and every rank must end with exactly the update a single process
computes from all N workers -- whatever the number of ranks and however unevenly N divides.
"""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

N, D, L = 5, 3001, 8


def _gradients():
    rng = np.random.default_rng(7)
    return (rng.standard_t(3.0, (N, D)) * 1e-3).astype(np.float32)


def _single_process(orc):
    g = _gradients()
    ps = [orc.params(orc.stats(g[i]), L, orc.NONUNIFORM, 3.0) for i in range(N)]
    rows = np.stack([orc.compress(g[i], ps[i], 42, i) for i in range(N)])
    return rows, orc.decompress_aggregate(rows, D, ps)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import ctypes
        import oracle as orc
        from paper_2402_01798_b200 import exchange
        g = _gradients()
        first, count = exchange.worker_slice(rank, world, N)
        mine = [orc.params(orc.stats(g[i]), L, orc.NONUNIFORM, 3.0) for i in range(first, first + count)]
        rows = [orc.compress(g[first + k], mine[k], 42, first + k) for k in range(count)]       # global worker index in the RNG
        words = orc.packed_words(D, 3)
        local_rows = torch.from_numpy(np.stack(rows).view(np.int32)) if count else torch.empty((0, words), dtype=torch.int32)
        size = ctypes.sizeof(orc.Params)
        local_par = torch.tensor(np.frombuffer(b"".join(bytes(p) for p in mine), dtype=np.uint8).reshape(count, size)
                                 if count else np.empty((0, size), dtype=np.uint8))
        all_rows = exchange.gather_worker_rows(local_rows, N).numpy().view(np.uint32)
        all_par = exchange.gather_worker_rows(local_par, N).numpy()
        ps = [orc.Params.from_buffer_copy(all_par[i].tobytes()) for i in range(N)]
        update = orc.decompress_aggregate(all_rows, D, ps)
        out[rank] = (all_rows.tobytes(), update.tobytes())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_workers_give_the_single_process_update(orc, world):
    port = 31000 + (os.getpid() * 7 + world) % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    rows, update = _single_process(orc)
    assert set(res) == set(range(world))
    for r in range(world):
        assert res[r][0] == rows.tobytes()            # every rank holds all N rows, in worker order
        assert res[r][1] == update.tobytes()          # and forms the same update, bit for bit


def test_worker_slices_tile_the_workers():
    from paper_2402_01798_b200 import exchange
    for world in (1, 2, 3, 4, 8):
        for n in (0, 1, 5, 8, 16, 63, 64):
            sl = exchange.all_worker_slices(world, n)
            assert sl[0][0] == 0 and sum(c for _, c in sl) == n
            for (f0, c0), (f1, _) in zip(sl, sl[1:]):
                assert f1 == f0 + c0
            counts = [c for _, c in sl]
            assert max(counts) - min(counts) <= 1
    with pytest.raises(ValueError):
        exchange.worker_slice(2, 2, 4)
