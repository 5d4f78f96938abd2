"""Seeded synthetic inputs and workload graph records (no operator arithmetic)."""
from . import gen, graphs  # noqa: F401
