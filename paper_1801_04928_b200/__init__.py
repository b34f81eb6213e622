"""B200 (sm_100a) library for the leapfrog backward pass of a sigmoid MLP (arXiv 1801.04928).

The work is done by hand-written CUDA kernels behind the C ABI of ``include/leapfrog.h``;
this package is the ctypes binding.  The shared library is loaded on first use of any name of
the binding and that fails loudly if it has not been built (``python -m
paper_1801_04928_b200.build``); there is no fallback.  ``paper_1801_04928_b200.build`` itself
can be imported without the library.
"""
import importlib

_BINDING = None


def _binding():
    global _BINDING
    if _BINDING is None:
        _BINDING = importlib.import_module(".binding", __name__)
    return _BINDING


def __getattr__(name):
    if name.startswith("__"):
        raise AttributeError(name)
    if name in ("build", "binding"):
        return importlib.import_module("." + name, __name__)
    try:
        return getattr(_binding(), name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
