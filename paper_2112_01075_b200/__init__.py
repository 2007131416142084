"""B200-native execution of synthesized array redistributions (after arXiv 2112.01075).

``api``        ctypes binding of the C boundary (``include/redist.h``); loads the CUDA library lazily
``workloads``  seeded synthetic meshes, types and global arrays (no method arithmetic)
``build``      nvcc build step for the library
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "api", "build"]


def __getattr__(name):
    if name in ("api", "build"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
