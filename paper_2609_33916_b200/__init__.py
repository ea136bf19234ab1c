"""B200-native fused attention forward+backward (sm_100a) behind a C-ABI library.

Importing the package is cheap and needs no GPU; the CUDA library is loaded the
first time a binding function is called (see `binding`).
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
