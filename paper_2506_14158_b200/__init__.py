"""B200-native verify step for S4C speculative decoding (arXiv 2506.14158).

``s4c``        thin ctypes binding over ``libs4c.so`` (the C-ABI CUDA library; all compute runs there)
``workloads``  seeded synthetic inputs (no method arithmetic)
``build``      in-tree nvcc build of ``libs4c.so`` for sm_100a
"""
from ._build import build, lib_path  # noqa: F401

__all__ = ["build", "lib_path", "s4c", "workloads"]


def __getattr__(name):
    if name in ("s4c", "workloads"):
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
