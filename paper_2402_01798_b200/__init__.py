"""B200-native truncated quantization of heavy-tailed gradients (TQSGD / TNQSGD hot path).

The product is ``libtq.so`` (hand-written sm_100a CUDA kernels behind a C ABI, declared in
``include/tq.h``).  This package is a thin binding with the same names: it marshals arguments,
nothing else -- every step of the path runs in the library.  PyTorch is used for device memory
and streams only.

``inputs`` (seeded synthetic gradients) can be imported without the library or a GPU; everything
in ``binding`` raises loudly when ``libtq.so`` is missing instead of falling back to anything.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
