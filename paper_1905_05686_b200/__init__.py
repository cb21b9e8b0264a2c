"""B200 (sm_100a) kernels for inference with a layer pruned by a tiled low-rank binary index.

``synth`` (inputs and packed formats, numpy only) imports without CUDA.  The
compute entry points live in ``binding`` and load the C-ABI library on first
use; they raise if the library has not been built -- there is no CPU fallback.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib

        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
