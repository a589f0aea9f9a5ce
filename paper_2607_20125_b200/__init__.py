"""HeadCast attention path for B200: ctypes binding over a hand-written CUDA (sm_100a) library.

``synth`` (seeded inputs) imports without CUDA; ``binding`` loads libheadcast.so on first use.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
