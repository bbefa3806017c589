"""The exchange variants of the round on ONE GPU as a one-rank NCCL group: the packed rows all-gathered, or left in
symmetric memory and read in place through their addresses by tq_decompress_aggregate_rows.  Both must produce
the same aggregated update (same parameter records, same rows, same worker order).  More than one GPU is needed
to move bytes between devices; this checks the plumbing and the row-address kernel path end to end."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def _run(mode):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29547", NCCL_NVLS_ENABLE="0")
    r = subprocess.run([sys.executable, "bench.py", "--config", "1", "--steps", "3", "--warmup", "3", "--exchange", mode],
                       cwd=ROOT, capture_output=True, text=True, timeout=900, env=env)
    return r


def test_allgather_and_peer_rows_give_the_same_update():
    a = _run("allgather")
    assert a.returncode == 0, a.stderr[-2000:]
    ja = json.loads([ln for ln in a.stdout.splitlines() if ln.startswith("{")][-1])
    p = _run("peer")
    if p.returncode != 0 and ("symmetric" in p.stderr.lower() or "symm" in p.stderr.lower()):
        pytest.skip("symmetric memory is not available on this box")
    assert p.returncode == 0, p.stderr[-2000:]
    jp = json.loads([ln for ln in p.stdout.splitlines() if ln.startswith("{")][-1])
    assert ja["config"]["workload"] == jp["config"]["workload"] == "resnet18-11.2M"
    assert ja["update_checksum"] == jp["update_checksum"] and ja["update_checksum"] != 0.0
    assert ja["gpu_launches"] > 0 and jp["gpu_launches"] > 0 and ja["scaling"] == "strong"
