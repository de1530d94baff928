"""B200-native fused 3D-RoPE attention (C-ABI library + thin Python binding).

Importing the package is cheap and needs no GPU; the CUDA shared library is
loaded on the first call into :mod:`paper_2607_28144_b200.binding` and a
missing library is a hard error (there is no CPU or library fallback).
"""
__all__ = ["binding", "synth"]
