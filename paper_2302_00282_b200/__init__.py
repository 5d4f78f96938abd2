"""Linked-chain CNN inference for B200 (sm_100a): Python binding of the C-ABI library."""
from . import binding  # noqa: F401
from .binding import Graph, HwInfo, XenosError, lib  # noqa: F401
