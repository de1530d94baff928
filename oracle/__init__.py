"""fp64 CPU oracle for the fused 3D-RoPE attention path.

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
CPU-baseline leg import this package.  It never imports the CUDA package.
"""
from .oracle import (  # noqa: F401
    PAIR_ADJACENT,
    PAIR_HALF,
    attn_core_head,
    attn_probs_row,
    brute_force,
    build,
    cross_attention,
    cross_attn_head,
    rope_angle,
    rope_freq,
    rope_pair,
    rope_rotate_f64,
    rope_rotate_head,
    rope_split,
    self_attention,
    self_attn_head,
    threads,
    token_position,
)
from . import qkv_oracle  # noqa: E402,F401
