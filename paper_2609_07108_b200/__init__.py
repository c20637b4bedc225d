"""Draft branch attention for B200 (sm_100a): packed variable-length main
sequences plus per-anchor draft branches (chain, block, tree), forward and
backward, with log-sum-exp merging of partial results over key chunks.

`workloads` holds the seeded synthetic input generators; `binding` is the thin
ctypes layer over the C-ABI CUDA library (imported lazily so that the
generators stay usable without the compiled library).
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
