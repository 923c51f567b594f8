"""FLuRKA attention forward pass (arxiv 2306.15799, Eq. (2)) as hand-written CUDA for sm_100a.

The compute lives in ``csrc/`` behind the C ABI declared in ``include/flurka.h``; ``binding``
is the thin ctypes layer with the same names.  Importing this package loads nothing native.
"""
from .configs import PERFORMER, RNN  # noqa: F401

__all__ = ["PERFORMER", "RNN"]
