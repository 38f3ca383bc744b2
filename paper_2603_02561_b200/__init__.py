"""B200-native SVD-Attention forward pass (SOLAR, arxiv 2603.02561).

`workloads` (seeded synthetic inputs) imports without the CUDA library; the
binding in `solar` loads the in-tree shared library on first use and raises
if it is missing -- there is no CPU fallback.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "solar"]


def __getattr__(name):
    if name == "solar":
        import importlib
        return importlib.import_module(".solar", __name__)
    raise AttributeError(name)
