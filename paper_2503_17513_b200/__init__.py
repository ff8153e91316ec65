"""B200-native expanded W4A4 linear layer (post-training model expansion, Sec. 3 of the paper).

``xq`` is the thin binding over the C-ABI CUDA library (loaded on first use; a missing
library is an error, there is no fallback).  ``synth`` draws the seeded synthetic inputs.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "xq"]


def __getattr__(name):
    if name == "xq":
        import importlib

        return importlib.import_module(".xq", __name__)
    raise AttributeError(name)
