"""Seeded synthetic inputs shaped like the decoder's windows.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only draws N(0, 1) numbers, applies the
stated per-head scale, rounds to bf16 and describes the five workloads.

The paper's talking-head clips are not public; these tensors stand in for the
query/key/value activations of one window: a latent token grid T x H x W
(4x8x8 VAE compression then 2x2 patchify of a 25-frame window), heads of
width 128, and the 512-token (T5) and 257-token (CLIP) conditioning
sequences whose per-layer key/value tensors the paper streams to the GPU
(Sec. 3.9).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np
import torch

HEAD_DIM = 128
ROPE_THETA = 10000.0

# generator streams
STREAM_Q, STREAM_K, STREAM_V, STREAM_CK, STREAM_CV, STREAM_SCALE, STREAM_X, STREAM_W, STREAM_B, STREAM_G = range(10)
STREAM_WO, STREAM_BO = 10, 11


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    T: int
    H: int
    W: int
    n_heads: int
    layers: int                      # transformer blocks per forward
    steps: int = 4                   # denoising steps per window
    cross_kv: Tuple[int, ...] = ()   # conditioning sequence lengths
    head_scale: Optional[Tuple[float, float]] = None  # U[lo, hi] per head on q, k, v
    head_dim: int = HEAD_DIM
    theta: float = ROPE_THETA

    @property
    def n_tokens(self) -> int:
        return self.T * self.H * self.W

    def self_flops(self) -> float:
        return 4.0 * self.n_heads * float(self.n_tokens) ** 2 * self.head_dim

    def cross_flops(self, n_kv: int) -> float:
        return 4.0 * self.n_heads * float(self.n_tokens) * n_kv * self.head_dim


WORKLOADS = {
    "tiny": Workload("tiny", 11, 2, 8, 8, 2, layers=1),
    "window_256x256": Workload("window_256x256", 12, 7, 16, 16, 12, layers=30),
    "window_480x832": Workload("window_480x832", 13, 7, 30, 52, 12, layers=30, cross_kv=(512,)),
    "large_480x832_ref": Workload("large_480x832_ref", 14, 8, 30, 52, 40, layers=40, head_scale=(0.5, 2.0)),
    "clip_77f": Workload("clip_77f", 15, 20, 30, 52, 40, layers=40, cross_kv=(512, 257)),
}
WORKLOAD_ORDER = ["tiny", "window_256x256", "window_480x832", "large_480x832_ref", "clip_77f"]


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) * 64 + int(stream))
    return g


def head_scales(seed: int, n_heads: int, lo: float, hi: float) -> torch.Tensor:
    u = torch.rand((n_heads,), generator=_gen(seed, STREAM_SCALE), dtype=torch.float32)
    return lo + (hi - lo) * u


def normal_bf16(seed: int, stream: int, n_tokens: int, n_heads: int, head_dim: int = HEAD_DIM,
                scales: Optional[torch.Tensor] = None) -> torch.Tensor:
    """[n_tokens, n_heads, head_dim] bf16 on the CPU: N(0,1) (times the head's scale), rounded RNE."""
    x = torch.randn((n_tokens, n_heads, head_dim), generator=_gen(seed, stream), dtype=torch.float32)
    if scales is not None:
        x.mul_(scales.view(1, n_heads, 1))
    return x.to(torch.bfloat16)


def self_inputs(w: Workload):
    """q, k, v for the self-attention call of workload ``w`` (CPU bf16)."""
    sc = head_scales(w.seed, w.n_heads, *w.head_scale) if w.head_scale else None
    q = normal_bf16(w.seed, STREAM_Q, w.n_tokens, w.n_heads, w.head_dim, sc)
    k = normal_bf16(w.seed, STREAM_K, w.n_tokens, w.n_heads, w.head_dim, sc)
    v = normal_bf16(w.seed, STREAM_V, w.n_tokens, w.n_heads, w.head_dim, sc)
    return q, k, v


def cross_inputs(w: Workload, n_kv: int):
    """k, v of one conditioning sequence (no rotation applies to them)."""
    k = normal_bf16(w.seed + 1000 * n_kv, STREAM_CK, n_kv, w.n_heads, w.head_dim)
    v = normal_bf16(w.seed + 1000 * n_kv, STREAM_CV, n_kv, w.n_heads, w.head_dim)
    return k, v


def block_inputs(w: Workload):
    """Inputs of the producer step in front of self-attention (the block's QKV projection): token features
    x [N, C] ~ N(0, 1) bf16, weights w_qkv [3C, C] ~ N(0, 1/C) bf16 (so that projected features are O(1), as after a
    normalisation layer), bias [3C] ~ N(0, 0.1^2) fp32, norm gains g_q, g_k [C] ~ U[0.5, 1.5] fp32, eps = 1e-6.
    Stand-ins for activations and trained weights, which are not available here."""
    C = w.n_heads * w.head_dim
    x = torch.randn((w.n_tokens, C), generator=_gen(w.seed, STREAM_X), dtype=torch.float32).to(torch.bfloat16)
    wq = (torch.randn((3 * C, C), generator=_gen(w.seed, STREAM_W), dtype=torch.float32) / C ** 0.5).to(torch.bfloat16)
    b = 0.1 * torch.randn((3 * C,), generator=_gen(w.seed, STREAM_B), dtype=torch.float32)
    g = 0.5 + torch.rand((2, C), generator=_gen(w.seed, STREAM_G), dtype=torch.float32)
    return x, wq, b, g[0].contiguous(), g[1].contiguous(), 1e-6


def out_proj_inputs(w: Workload):
    """Inputs of the block's output projection: weights w_o [C, C] ~ N(0, 1/C) bf16 and bias [C] ~ N(0, 0.1^2) fp32
    (stand-ins for trained weights, like block_inputs)."""
    C = w.n_heads * w.head_dim
    wo = (torch.randn((C, C), generator=_gen(w.seed, STREAM_WO), dtype=torch.float32) / C ** 0.5).to(torch.bfloat16)
    bo = 0.1 * torch.randn((C,), generator=_gen(w.seed, STREAM_BO), dtype=torch.float32)
    return wo, bo


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 CPU tensor -> uint16 bit patterns (what the oracle takes)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_f32(a) -> torch.Tensor:
    """Any float array -> bf16 CPU tensor (round to nearest even)."""
    return torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)


def sample_rows(n_tokens: int, H: int, W: int, seed: int, n_random: int = 256) -> np.ndarray:
    """Query rows worth checking at the large shapes: the first tile, the whole
    ragged tail tile, both sides of the 128/256-row boundaries around the
    middle, the rows where y or x wrap, and seeded random rows."""
    rows = set(range(min(128, n_tokens)))
    tail0 = (n_tokens - 1) // 128 * 128
    rows.update(range(tail0, n_tokens))
    mid = (n_tokens // 2) // 256 * 256
    for b in (mid - 256, mid - 128, mid, mid + 128, mid + 256):
        for r in (b - 2, b - 1, b, b + 1):
            if 0 <= r < n_tokens:
                rows.add(r)
    for r in (W - 1, W, H * W - 1, H * W, 2 * H * W - 1, 2 * H * W):
        if 0 <= r < n_tokens:
            rows.add(r)
    rng = np.random.Generator(np.random.Philox(key=seed))
    rows.update(int(r) for r in rng.integers(0, n_tokens, size=n_random))
    return np.array(sorted(rows), dtype=np.int64)
