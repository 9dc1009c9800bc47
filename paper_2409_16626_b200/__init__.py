"""B200-native HiFloat8 (HiF8) conversion library: thin Python binding over the C ABI in include/hif8.h.

The binding (and with it libhif8.so) is loaded on first attribute access, so that
`python -m paper_2409_16626_b200.build` can run before the library exists.
"""
import importlib

_SUBMODULES = ("build", "binding", "sharded")


def __getattr__(name):
    if name in _SUBMODULES:
        return importlib.import_module("." + name, __name__)
    binding = importlib.import_module(".binding", __name__)
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
