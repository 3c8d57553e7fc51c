"""B200 (sm_100a) hot path of SplitBrain hybrid data/model-parallel CNN training.

The product is the C-ABI shared library built from csrc/ (declared in include/splitbrain.h);
`binding` is a thin ctypes layer with the same entry-point names.  It is imported on first use, so
that `python -m paper_2112_15317_b200.build_ext` can build the library before it exists; using
`binding`, `Model` or `SBError` without the built library raises ImportError (there is no fallback).
"""
import importlib

__all__ = ["binding", "Model", "SBError"]


def __getattr__(name):
    if name == "binding":
        return importlib.import_module(".binding", __name__)
    if name in ("Model", "SBError"):
        return getattr(importlib.import_module(".binding", __name__), name)
    raise AttributeError(name)
