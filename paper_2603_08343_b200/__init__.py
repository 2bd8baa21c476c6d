"""B200 (sm_100a) Walsh-Hadamard head mixing with a diagonal affine.

    y = a (.) (x H_d)/sqrt(d) + b        on every row of x[T, d]

The compute lives in a C-ABI shared library (csrc/, include/wht_affine.h) made of
hand-written CUDA kernels; `binding` is a thin ctypes layer with the same entry
point names.  The library is loaded on first use and a missing or unloadable
library raises: there is no CPU fallback.
"""
from . import workloads  # noqa: F401


_SUBMODULES = ("binding", "build", "dp", "tp", "autograd", "workloads")


def __getattr__(name):
    # The binding (and with it the shared library) is loaded lazily so that input generation and
    # the build step can be imported on machines without the built library.
    import importlib
    if name in _SUBMODULES:
        return importlib.import_module("." + name, __name__)
    if name.startswith("__"):
        raise AttributeError(name)
    _b = importlib.import_module(".binding", __name__)
    if hasattr(_b, name):
        return getattr(_b, name)
    raise AttributeError(name)
