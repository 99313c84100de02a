"""HCCS (Head-Calibrated Clipped-Linear Softmax) inference kernels for NVIDIA B200.

``workloads`` (numpy only) can be imported anywhere; everything else needs the
compiled CUDA library ``csrc/libhccs.so`` and raises if it is missing.
"""
import importlib

from . import workloads  # noqa: F401

__all__ = ["workloads"]
_SUBMODULES = ("build", "binding")


def __getattr__(name):
    # The binding is loaded on first use so that the input generators work on hosts without
    # the compiled library; a missing library is an ImportError, never a fallback.
    if name.startswith("__"):
        raise AttributeError(name)
    if name in _SUBMODULES:                  # `from package import build` must work before the library exists
        return importlib.import_module(__name__ + "." + name)
    binding = importlib.import_module(__name__ + ".binding")
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
