"""B200 (sm_100a) hot path of SplitBrain hybrid data/model-parallel CNN training.

The product is the C-ABI shared library built from csrc/ (declared in include/splitbrain.h);
`binding` is a thin ctypes layer with the same entry-point names.
"""
from . import binding  # noqa: F401
from .binding import Model, SBError  # noqa: F401
