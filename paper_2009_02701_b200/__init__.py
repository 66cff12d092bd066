"""HPSGD replica update + delayed merge on one B200: ctypes binding of ``libhpsgd.so``.

The CUDA library is the only implementation; importing :mod:`binding` does not load it,
the first call does, and that call fails loudly if the library has not been built.
"""
from . import binding   # noqa: F401
from .binding import *  # noqa: F401,F403
