"""Seeded synthetic inputs and workload definitions (no HPSGD arithmetic)."""
from . import hashgen            # noqa: F401
from .configs import Layout, Workload, get, names   # noqa: F401
