"""SAGE-KV hot path (arXiv 2503.08879, Section 2) as sm_100a CUDA kernels.

`paper_2503_08879_b200.binding` is the thin ctypes layer over the C-ABI library
(include/sagekv.h); `paper_2503_08879_b200.synth` draws the seeded synthetic
inputs.  Importing the binding fails loudly if the library has not been built.
"""

__all__ = ["synth"]
