"""Dependency-masked multi-branch decode attention for B200 (sm_100a).

`workloads` holds the seeded synthetic inputs; `fdc` is the thin ctypes binding of the
C-ABI CUDA library (loaded on first use; it raises if the library has not been built)."""
from . import workloads  # noqa: F401

__all__ = ["workloads", "fdc"]


def __getattr__(name):
    if name == "fdc":
        import importlib
        return importlib.import_module(__name__ + ".fdc")
    raise AttributeError(name)
