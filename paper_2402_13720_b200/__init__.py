"""Ouroboros verification path for one B200: CUDA library (libouro.so) plus a thin ctypes binding."""
from . import synth  # noqa: F401
from .binding import Engine, OuroError, lib  # noqa: F401
