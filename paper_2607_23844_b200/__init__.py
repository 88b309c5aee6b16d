"""B200-native OmniCache hot path: match / select / gather / restore / layered cache.

The CUDA work lives in ``csrc/`` behind a C-ABI shared library (``include/omnicache.h``);
``omnicache`` is the thin ctypes binding over it.  ``inputs`` draws the seeded synthetic tensors.
Submodules are imported lazily so that drawing inputs never needs the compiled library.
"""
import importlib

__all__ = ["omnicache", "inputs", "build", "sharding"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
