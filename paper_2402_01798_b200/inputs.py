"""Seeded synthetic heavy-tailed gradients.

This module only makes INPUT DATA.  It holds none of the compressor's arithmetic
(no truncation, rounding, packing, statistics or parameter formulas) and is the one
piece of code that both the CUDA library's tests/benchmarks and the CPU oracle's tests
may use.  It imports neither of them.

The paper's workloads are flat gradients of convolutional/fully-connected networks whose
element density has a power-law tail (Section 4.1, the power-law definition and the
tail model that follows it).  Those gradients are not available offline, so seeded
synthetic vectors with the same shape stand in: element magnitudes follow a Lomax
law, ``|g| = scale * ((1 - U)^(-1/(gamma-1)) - 1)`` with ``U ~ Uniform[0,1)``, whose
density is proportional to ``(1 + x/scale)^(-gamma)`` (tail exponent ``gamma`` in the
paper's convention), the sign is a fair coin, and elements are independent (the
assumption stated before Lemma 2).  Optionally a Bernoulli(``outlier_frac``) subset is
multiplied by ``outlier_mult`` and the result is stored as bfloat16.

Everything is drawn from a ``torch.Generator`` seeded by the caller, on the device the
caller names, in bounded chunks, so a 10^9-element vector never needs more than a few
hundred MB of scratch.  CPU and CUDA generators give different streams; parity tests
therefore always hand the oracle the very bytes the GPU consumed.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple

import torch

_CHUNK = 1 << 25  # elements generated per step (128 MB of fp32 scratch per temporary)


def powerlaw_gradient(
    d: int,
    gamma: float,
    scale: float,
    seed: int,
    device: str | torch.device = "cpu",
    dtype: torch.dtype = torch.float32,
    outlier_frac: float = 0.0,
    outlier_mult: float = 100.0,
    out: Optional[torch.Tensor] = None,
) -> torch.Tensor:
    """Fill (or allocate) a length-``d`` vector with seeded Lomax-magnitude, random-sign values."""
    if gamma <= 1.0:
        raise ValueError("gamma must exceed 1")
    device = torch.device(device)
    if out is None:
        out = torch.empty(d, dtype=dtype, device=device)
    if out.numel() != d or out.dtype != dtype:
        raise ValueError("out has the wrong size or dtype")
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    expo = -1.0 / (gamma - 1.0)
    for lo in range(0, d, _CHUNK):
        n = min(_CHUNK, d - lo)
        u = torch.rand(n, generator=gen, device=device, dtype=torch.float32)
        mag = (1.0 - u).pow_(expo).sub_(1.0).mul_(scale)
        sgn = torch.rand(n, generator=gen, device=device, dtype=torch.float32)
        mag = torch.where(sgn < 0.5, -mag, mag)
        if outlier_frac > 0.0:
            pick = torch.rand(n, generator=gen, device=device, dtype=torch.float32)
            mag = torch.where(pick < outlier_frac, mag * outlier_mult, mag)
        out[lo:lo + n].copy_(mag)  # rounds to nearest-even when dtype is bfloat16
    return out


@dataclass(frozen=True)
class Workload:
    """One of the benchmark configurations: shape, distribution and quantizer choice."""
    name: str
    d: int
    n_workers: int
    gamma: float
    scale: float
    mode: str            # "uniform" | "nonuniform"
    num_levels: int      # L = 2^bits quantization points
    dtype: torch.dtype = torch.float32
    outlier_frac: float = 0.0
    outlier_mult: float = 100.0
    base_seed: int = 0
    note: str = ""

    @property
    def bits(self) -> int:
        return {2: 1, 4: 2, 8: 3, 16: 4}[self.num_levels]


def _cfg4(gamma: float, mode: str, levels: int) -> Workload:
    return Workload(
        name=f"gpt2s-124M-bf16-g{gamma}-{mode}-L{levels}", d=124_000_000, n_workers=8,
        gamma=gamma, scale=1e-4, mode=mode, num_levels=levels, dtype=torch.bfloat16,
        outlier_frac=0.01, outlier_mult=100.0, base_seed=4000,
        note="bf16 storage, upcast in-kernel; 1% of entries are 100x outliers")


WORKLOADS = {
    # index -> the five benchmark configurations (config 3 is a 12-case sweep; its
    # canonical member is gamma=3, non-uniform, L=16; the others are in CONFIG4_SWEEP)
    0: Workload("tiny-100k", 100_000, 1, 3.0, 1e-3, "uniform", 4, base_seed=0),
    1: Workload("resnet18-11.2M", 11_200_000, 8, 2.5, 1e-3, "uniform", 8, base_seed=1000),
    2: Workload("resnet50-25.6M", 25_600_000, 16, 3.0, 5e-4, "nonuniform", 16, base_seed=2000),
    3: _cfg4(3.0, "nonuniform", 16),
    4: Workload("flat-1e9", 1_000_000_000, 4, 2.5, 1e-4, "nonuniform", 8, base_seed=5000),
}

CONFIG4_SWEEP = tuple(
    _cfg4(g, m, L) for g in (2.2, 3.0, 4.0) for m in ("uniform", "nonuniform") for L in (4, 16)
)


def worker_stride(d: int, dtype: torch.dtype) -> int:
    """Elements between consecutive workers' slices: d rounded up so every slice starts 32-byte aligned."""
    per = 32 // torch.empty((), dtype=dtype).element_size()
    return (d + per - 1) // per * per


def make_worker_gradients(w: Workload, device: str | torch.device,
                          d: Optional[int] = None) -> Tuple[torch.Tensor, int]:
    """All workers' gradients as one ``[N, stride]`` tensor (worker i is seeded ``base_seed + i``).

    Returns the tensor and the stride in elements.  Padding elements (when ``d`` is not a
    multiple of the alignment unit) are zero and are never read by the library.
    """
    d = w.d if d is None else d
    stride = worker_stride(d, w.dtype)
    g = torch.zeros((w.n_workers, stride), dtype=w.dtype, device=device)
    for i in range(w.n_workers):
        powerlaw_gradient(d, w.gamma, w.scale, w.base_seed + i, device, w.dtype,
                          w.outlier_frac, w.outlier_mult, out=g[i, :d])
    return g, stride
