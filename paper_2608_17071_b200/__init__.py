"""kx: BF16 attention output projection with residual addition for B200 (sm_100a).

``Y = X W^T (+ bias) + R`` and the plain GEMM, as hand-written tcgen05 / TMA
kernels behind a C ABI (``include/kx.h``).  This package holds the CUDA sources
(``csrc/``), the build step (``build``), the ctypes binding (``binding``) and the
seeded input generator (``inputs``).  Importing the package does not load the
CUDA library; the binding's functions do, and raise if it is missing.
"""
from importlib import import_module as _im

__all__ = ["binding", "build", "inputs"]


def __getattr__(name):
    if name in __all__:
        return _im(f"{__name__}.{name}")
    b = _im(f"{__name__}.binding")
    if hasattr(b, name):
        return getattr(b, name)
    raise AttributeError(name)
