"""B200-native SemantiCache hot path: chunk -> GSC -> merge -> proportional-attention decode.

The compute lives in hand-written sm_100a CUDA kernels behind a C-ABI library
(``include/semanticache.h``); :mod:`.binding` marshals torch device tensors into those
calls and :mod:`.synth` draws the seeded synthetic workloads.  Importing the package
loads nothing; the first call into :mod:`.binding` loads the library and raises if it
has not been built (there is no CPU fallback).
"""
__all__ = ["binding", "synth", "build"]
