"""Delayed synchronous step of ABS-SGD (arXiv 2308.15164, Algorithm 1) on one B200.

The package holds three things:

* ``csrc/``      -- the sm_100a CUDA kernels and the C-ABI library built from them
                   (entry points declared in ``include/abs_sgd.h``),
* ``binding``    -- a ctypes binding with the same names (argument marshalling only),
* ``workloads``  -- seeded synthetic input generators (no optimiser arithmetic).

Nothing here falls back to a CPU implementation: importing ``binding`` raises if the
shared library has not been built.
"""

__all__ = ["binding", "workloads", "build", "dist"]


def __getattr__(name):
    # Lazy sub-module import so that ``workloads`` can be used without the CUDA library.
    if name in __all__:
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
