"""B200-native decode hot path of SeerAttention-R: AttnGate scoring over a compressed-K
cache, token-budget block selection, block-sparse GQA split-KV flash decoding.

The work is done by hand-written sm_100a CUDA kernels behind a C-ABI shared library
(``include/seer.h``); :mod:`paper_2506_08889_b200.binding` is the thin ctypes layer over
it and raises at first use if the library has not been built (there is no CPU fallback).
:mod:`paper_2506_08889_b200.synth` draws the seeded synthetic workloads.
"""
__all__ = ["binding", "synth", "build"]
