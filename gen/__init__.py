"""Seeded synthetic input generators (no cache arithmetic lives here)."""
from . import workloads  # noqa: F401
