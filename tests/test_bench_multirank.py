"""The N > 1 path of bench.py on CPU: two gloo ranks.

On several GPUs every rank runs its own replica of the workload (own seeds) and the only thing that
crosses ranks is the timing: the slowest rank's time divides the work of all ranks.  This test runs
that logic with world_size = 2 over gloo, without a GPU.
"""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        from paper_2402_01798_b200 import inputs
        w = bench.replica_workload(inputs.WORKLOADS[0], rank)
        g, _ = inputs.make_worker_gradients(w, "cpu", d=4096)
        my_ms = 2.0 + 3.0 * rank                                  # rank 1 is the slow one
        dist.barrier()
        ms = bench.max_over_ranks(my_ms, world)
        value = bench.whole_job_gbs(world, 4096 * 4, ms)
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, g.double().abs().sum().reshape(1))
        out[rank] = (ms, value, w.base_seed, [float(x) for x in sums])
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        ms, value, seed, sums = res[rank]
        assert ms == 5.0                                          # max over ranks, identical on both
        assert value == pytest.approx(2 * 4096 * 4 / 5.0e-3 / 1e9)
    assert res[0][2] != res[1][2]                                 # replicas: different seeds ...
    assert res[0][3][0] != res[0][3][1]                           # ... and different data
    assert res[0][3] == res[1][3]


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.whole_job_gbs(1, 10**9, 1000.0) == 1.0
