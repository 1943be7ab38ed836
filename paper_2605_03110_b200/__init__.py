"""B200-native Gram-threshold representative-token selection (Cascade ADA hot path).

`workloads` (seeded synthetic inputs) imports without the CUDA library;
everything else goes through `binding`, which loads the in-tree C-ABI shared
library and raises if it has not been built -- there is no CPU fallback.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
