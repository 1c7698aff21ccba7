"""LiteVAR multi-diagonal windowed attention for B200 (sm_100a).

The compute path lives in the C-ABI shared library built from ``csrc/`` and is reached
through :mod:`paper_2411_17178_b200.binding`.  Importing the package does not load the
library; the first call that needs it does, and raises if it has not been built.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
