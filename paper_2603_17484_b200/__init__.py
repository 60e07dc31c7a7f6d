"""B200-native (sm_100a) hot path of the L2A conditional attention layer.

``l2a`` holds the thin binding over the C-ABI library (``libl2a.so``); ``synth`` holds the seeded
synthetic input generators.  Importing the package does not load the CUDA library; the first call
into ``l2a`` does, and fails loudly if it has not been built.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "l2a"]


def __getattr__(name):
    if name == "l2a":
        import importlib
        return importlib.import_module(".l2a", __name__)
    raise AttributeError(name)
