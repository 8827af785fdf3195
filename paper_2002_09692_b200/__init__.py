"""SAPS-PSGD gossip round for NVIDIA B200: ctypes binding of the CUDA library.

``from paper_2002_09692_b200 import binding`` loads ``libsaps.so`` (built in-tree by
``python -m paper_2002_09692_b200.build``); ``synth`` holds the seeded input generators.
The binding is imported on first use so that the input generators can be used on their own.
"""
import importlib

__all__ = ["binding", "synth", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
