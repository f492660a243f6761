"""Sparse tensor kernels over per-level (dense | compressed) storage for B200.

``paper_2202_04305_b200.binding`` is the Python face of the C ABI in
``include/sp.h`` (it needs the built ``libsp.so`` and a CUDA device);
``paper_2202_04305_b200.inputs`` holds the seeded synthetic input recipes.
Submodules are imported on first use so that the input recipes stay usable
on a machine without the CUDA library.
"""
import importlib

__all__ = ["binding", "inputs", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
