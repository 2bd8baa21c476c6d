"""B200 (sm_100a) Walsh-Hadamard head mixing with a diagonal affine.

    y = a (.) (x H_d)/sqrt(d) + b        on every row of x[T, d]

The compute lives in a C-ABI shared library (csrc/, include/wht_affine.h) made of
hand-written CUDA kernels; `binding` is a thin ctypes layer with the same entry
point names.  The library is loaded on first use and a missing or unloadable
library raises: there is no CPU fallback.
"""
from . import workloads  # noqa: F401


def __getattr__(name):
    # The binding (and with it the shared library) is loaded lazily so that
    # input generation can be imported on machines without the built library.
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    from . import binding as _b
    if hasattr(_b, name):
        return getattr(_b, name)
    raise AttributeError(name)
