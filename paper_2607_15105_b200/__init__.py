"""B200-native (sm_100a) Hierarchical Global Attention hot path: summaries, routing,
routed exact-token attention forward and backward, behind a C-ABI shared library.

`workloads` draws the seeded synthetic inputs; `binding` marshals arguments into the
C-ABI calls (it loads the CUDA library on first use and fails loudly if it is missing).
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
