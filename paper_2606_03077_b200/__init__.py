"""B200-native paged GQA decode attention (planner + split-KV decode + combine).

``workloads`` (seeded input generators, NumPy only) can be imported without the CUDA
library; everything else lives in ``binding`` and raises at import time if the shared
library has not been built.
"""
__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
