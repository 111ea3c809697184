"""B200-native hot path of ZCCL: fZ-light codec, fused reduce-scatter hop, emulated ring collectives.

``fields`` holds the seeded synthetic inputs; ``zccl`` is the binding over the C-ABI library (imported lazily so
that input generation does not need torch or a GPU).
"""
import importlib

from . import fields  # noqa: F401

__all__ = ["fields", "zccl", "build"]


def __getattr__(name):
    if name in ("zccl", "build"):
        return importlib.import_module(f".{name}", __name__)
    raise AttributeError(name)
