"""B200-native sparse-MoE verify layer: hand-written sm_100a kernels behind a C ABI.

``workloads`` (seeded synthetic inputs) imports nothing else; the binding in ``api`` loads
the CUDA library on first use and raises if it is missing -- there is no CPU fallback.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "api"]


def __getattr__(name):
    if name == "api":
        import importlib

        return importlib.import_module(".api", __name__)
    raise AttributeError(name)
