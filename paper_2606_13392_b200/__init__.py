"""B200-native forward hot path of MiniMax Sparse Attention (MSA).

Three stages (Algorithm 1, lines 3-5): index scoring with block max-pool (Eq. 6),
exp-free Top-k block selection with the local block forced in (Eq. 7), and exact
block-sparse GQA attention over the selected blocks (Eq. 8), for prefill and decode.

The arithmetic lives in hand-written sm_100a CUDA kernels behind a C ABI
(``include/msa.h``); :mod:`paper_2606_13392_b200.binding` only marshals arguments.
Importing this package does not load the CUDA library; the first call does, and it
raises if the library is missing (there is no CPU fallback).
"""

from .inputs import MSAConfig, CONFIGS  # noqa: F401

__all__ = ["MSAConfig", "CONFIGS"]
