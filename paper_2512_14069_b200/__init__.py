"""B200-native hot path of one RADAR speculative step (C-ABI library + thin binding).

Importing the package loads nothing heavy: the CUDA library is opened on first
use of `paper_2512_14069_b200.binding`, and fails loudly if it is missing.
"""
__all__ = ["binding", "workloads"]
