"""B200 (sm_100a) implementation of the randomized-matrix-multiplication linear layer
of arXiv 2201.13195: a C-ABI CUDA library (include/rmm.h) and its ctypes binding.

The binding (and with it librmm.so) is loaded on first use of any attribute, so that
``python -m paper_2201_13195_b200.build`` can run before the library exists.  There is
no non-CUDA path: using the package without a built library raises ImportError.
"""
import importlib


_SUBMODULES = ("build", "binding")


def __getattr__(name):
    if name in _SUBMODULES:          # `from package import build` must work before the library exists
        return importlib.import_module("." + name, __name__)
    binding = importlib.import_module(".binding", __name__)
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
