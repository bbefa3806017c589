"""Writes tests/golden/oracle_small_case.txt: checksums of the ORACLE's outputs on a small seeded case.

Calls only oracle/ (never the CUDA library).  The file guards the oracle against accidental changes of
its arithmetic: a deliberate change regenerates it and says why in the commit message.

    python tests/golden/make_oracle_golden.py
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_small_case.txt")
CASES = [  # name, d, n_workers, gamma, scale, mode, levels
    ("uniform-L4", 100_000, 1, 3.0, 1e-3, oracle.UNIFORM, 4),
    ("uniform-L8", 50_003, 3, 2.5, 1e-3, oracle.UNIFORM, 8),
    ("nonuniform-L16", 50_003, 3, 3.0, 5e-4, oracle.NONUNIFORM, 16),
    ("biscaled-L8", 30_001, 2, 3.5, 1e-4, oracle.BISCALED, 8),
]


def gradient(d, gamma, scale, seed):
    """Lomax magnitudes with random signs from NumPy's PCG64 (stable across platforms)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    u = rng.random(d)
    mag = scale * ((1.0 - u) ** (-1.0 / (gamma - 1.0)) - 1.0)
    return (mag * np.where(rng.random(d) < 0.5, -1.0, 1.0)).astype(np.float32)


def digest(a):
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()[:32]


def lines():
    out = ["# case  alpha[worker 0] (hex)  sha256/128 of: levels, packed rows, aggregate"]
    for name, d, n, gamma, scale, mode, levels in CASES:
        ps, rows = [], []
        for i in range(n):
            g = gradient(d, gamma, scale, 7000 + i)
            st = oracle.stats(g)
            p = oracle.params(st, levels, mode, gamma)
            ps.append(p)
            rows.append(oracle.compress(g, p, 12345, i))
        packed = np.stack(rows)
        agg = oracle.decompress_aggregate(packed, d, ps)
        lv = np.concatenate([p.levels_np() for p in ps])
        out.append(f"{name} {float(ps[0].alpha).hex()} {digest(lv)} {digest(packed)} {digest(agg)}")
    return out


if __name__ == "__main__":
    with open(OUT, "w") as f:
        f.write("\n".join(lines()) + "\n")
    print(open(OUT).read())
