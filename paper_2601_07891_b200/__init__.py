"""KVzap pruning hot path for B200 (sm_100a): thin Python binding over the
C-ABI CUDA library in ``csrc/`` plus the seeded synthetic-input generators.

The CUDA library is loaded on first use (``paper_2601_07891_b200.binding``);
there is no CPU fallback: a missing or unbuilt library raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth"]
