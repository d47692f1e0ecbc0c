"""Seeded synthetic inputs for the SpecAttn verification hot path.

This package only manufactures inputs (probability rows, queries, paged K/V
pools, block tables, layer maps) with the shapes and value laws of the five
benchmark configurations.  It holds none of the method's arithmetic and is the
only code shared by the CPU oracle's tests and the CUDA library's tests.
"""
from . import bf16  # noqa: F401
from .generators import *  # noqa: F401,F403
from .configs import *  # noqa: F401,F403
