"""Pins for the oracle's random-bit source (reading R9 in oracle/tq_oracle.c).

The oracle's Philox4x32-10 is checked against things that are not the oracle:
  * the generator's published known-answer vectors (tests/golden/philox4x32_10_kat.txt);
  * an independent implementation: the Philox engine header that ships with PyTorch,
    compiled into a tiny program here and driven through its public interface;
  * statistics of the 16-bit slots the compressor consumes.
"""
import os
import subprocess
import sys

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat_rows():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[:4], w[4:6], w[6:]))
    return rows


def test_known_answer_vectors(orc):
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = orc.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == want


_TORCH_PROBE = r"""
#include <ATen/core/PhiloxRNGEngine.h>
#include <cstdio>
#include <cstdlib>
int main(int argc, char** argv) {
  // argv: triples (seed subsequence offset); prints the 4 words of that 128-bit block
  for (int i = 1; i + 2 < argc; i += 3) {
    unsigned long long seed = strtoull(argv[i], 0, 10), sub = strtoull(argv[i+1], 0, 10),
                       off = strtoull(argv[i+2], 0, 10);
    at::Philox4_32 eng(seed, sub, off);
    unsigned a = eng(), b = eng(), c = eng(), d = eng();
    printf("%u %u %u %u\n", a, b, c, d);
  }
  return 0;
}
"""


@pytest.fixture(scope="module")
def torch_philox_probe(tmp_path_factory):
    import torch
    inc = os.path.join(os.path.dirname(torch.__file__), "include")
    if not os.path.exists(os.path.join(inc, "ATen", "core", "PhiloxRNGEngine.h")):
        pytest.skip("this PyTorch build does not ship the Philox engine header")
    d = tmp_path_factory.mktemp("philox_probe")
    src, exe = d / "probe.cpp", d / "probe"
    src.write_text(_TORCH_PROBE)
    r = subprocess.run(["g++", "-O1", "-std=c++17", f"-I{inc}", str(src), "-o", str(exe)],
                       capture_output=True, text=True)
    if r.returncode != 0:
        pytest.skip("could not compile against the PyTorch Philox header: " + r.stderr[-300:])
    return str(exe)


def test_against_pytorch_engine(orc, torch_philox_probe):
    """Same (key, counter) -> same 128 bits as PyTorch's engine.

    That engine takes (seed, subsequence, offset): the seed is the key, the offset counts
    128-bit blocks (counter words 0-1) and the subsequence fills counter words 2-3.  The
    compressor's counter (j >> 3, worker) is therefore (offset = j >> 3, subsequence = worker).
    """
    rng = np.random.default_rng(7)
    cases = [(0, 0, 0), (1, 0, 0), (0, 1, 0), (0, 0, 1), (2**64 - 1, 2**32 - 1, 2**40 + 5)]
    for _ in range(40):
        cases.append((int(rng.integers(0, 2**63)) * 2 + int(rng.integers(0, 2)),
                      int(rng.integers(0, 2**32)), int(rng.integers(0, 2**48))))
    args = [str(x) for c in cases for x in c]
    out = subprocess.run([torch_philox_probe] + args, capture_output=True, text=True, check=True).stdout
    lines = out.strip().splitlines()
    assert len(lines) == len(cases)
    for (seed, worker, block), line in zip(cases, lines):
        want = [int(x) for x in line.split()]
        got = orc.philox4x32_10([block & 0xFFFFFFFF, block >> 32, worker, 0],
                                [seed & 0xFFFFFFFF, seed >> 32])
        assert [int(x) for x in got] == want, (seed, worker, block)


def test_slot_mapping(orc):
    """Element j reads 16-bit slot j & 7 of block j >> 3: slot q is the low (q even) or high (q odd)
    half of output word q >> 1.  Checked by rebuilding the 128-bit block from the eight slots."""
    seed, worker = 0x0123456789ABCDEF, 5
    for block in (0, 1, 77, 2**29 + 3, 2**33 + 11):
        words = orc.philox4x32_10([block & 0xFFFFFFFF, block >> 32, worker, 0],
                                  [seed & 0xFFFFFFFF, seed >> 32])
        big = sum(int(w) << (32 * i) for i, w in enumerate(words))
        for slot in range(8):
            j = block * 8 + slot
            assert orc.rand16(seed, worker, j) == (big >> (16 * slot)) & 0xFFFF


def test_slots_are_uniform_and_distinct_across_workers(orc):
    n = 1 << 16
    seed = 42
    r = np.array([[orc.rand16(seed, w, j) for j in range(n)] for w in (0, 1)], dtype=np.int64)
    for w in (0, 1):
        assert abs(r[w].mean() / 65535.0 - 0.5) < 4 * (1 / np.sqrt(12 * n))
        hist = np.bincount(r[w] >> 8, minlength=256)
        chi2 = ((hist - n / 256) ** 2 / (n / 256)).sum()
        assert chi2 < 255 + 6 * np.sqrt(2 * 255)          # about +6 sigma
    # different workers / different seeds give unrelated streams
    assert np.mean(r[0] == r[1]) < 5e-4
    r2 = np.array([orc.rand16(seed + 1, 0, j) for j in range(4096)])
    assert np.mean(r2 == r[0][:4096]) < 5e-3
    # adjacent slots are uncorrelated
    a, b = r[0][:-1] - 32767.5, r[0][1:] - 32767.5
    assert abs((a * b).mean() / (a.std() * b.std())) < 5 / np.sqrt(n)
