"""B200-native step executor for the Sparbit allgather (arXiv 2109.08751).

The package is a thin ctypes binding over libsparbit_b200.so (see include/sparbit.h).  Build the
library in-tree with `python -m paper_2109_08751_b200.build`.

The binding is loaded on first use of any of its names, so that the build module can be imported
before the library exists.  There is no fallback: using the package without the built library
raises ImportError.
"""
import importlib

_binding = None


def __getattr__(name):
    global _binding
    if name.startswith("__"):
        raise AttributeError(name)
    if name in ("build", "binding", "multi"):  # submodules
        return importlib.import_module("." + name, __name__)
    if _binding is None:
        _binding = importlib.import_module(".binding", __name__)
    try:
        return getattr(_binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
