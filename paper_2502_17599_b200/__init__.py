"""B200-native MEDA prefill KV-compression pass (arXiv 2502.17599): C-ABI CUDA library + thin binding.

`workloads` (synthetic input generators) imports without the compiled library; everything in
`binding` needs `libmeda.so` and raises if it is missing.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
