"""fp64 oracle of the producer step in front of the attention path -- TEST INFRASTRUCTURE, not product code.

The paper takes its transformer backbone by reference (Sec. 3.2 and 3.4 name the pose-controlled video diffusion
model it distils); in that published block the attention inputs are made from the token features x [N, C],
C = n_heads * head_dim, as

    y_q = x W_q^T + b_q,   y_k = x W_k^T + b_k,   v = x W_v^T + b_v          (three linear maps, C -> C)
    q   = y_q * g_q / sqrt(mean_c(y_q[c]^2) + eps)                           (RMS norm over ALL C features of a token)
    k   = y_k * g_k / sqrt(mean_c(y_k[c]^2) + eps)
    heads = consecutive blocks of head_dim features; the 3D rotary embedding then turns q and k of every head.

Written out here exactly in that order with numpy in fp64 (the matrix product is the library's, everything else
is element-wise); the rotation and the attention itself are the C oracle's.  Nothing is rounded on the way, so a
GPU path that fuses these steps into the projection's epilogue is compared with the unrounded result.

The weights are stored the way a linear layer stores them: w_qkv [3C, C], row f holds the weights of output
feature f; rows 0..C-1 make y_q, C..2C-1 make y_k, 2C..3C-1 make v.  b_qkv [3C], g_q, g_k [C].

The step behind the attention in the same block is its output projection: the heads' outputs of a token, laid side
by side as one row of C features (head a in features a*head_dim ...), go through one more linear map,

    y = o W_o^T + b_o                                                         (C -> C),

written out in `out_project`; `attention_block` chains all three steps without rounding anything in between.
"""
from __future__ import annotations

import numpy as np

from . import oracle as _o


def bf16_to_f64(bits) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64, exactly (a bf16 is the upper half of a binary32)."""
    bits = np.ascontiguousarray(bits)
    if bits.dtype != np.uint16:
        raise TypeError("bf16 tensors are passed as uint16 bit patterns")
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rms_norm(y: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y [N, C] -> y * g / sqrt(mean over the C features of y^2 + eps), row by row."""
    ms = (y * y).mean(axis=1, keepdims=True)
    return y * g[None, :] / np.sqrt(ms + eps)


def qkv_project(x_bits, w_bits, b, g_q, g_k, eps: float, n_heads: int):
    """x [N, C], w_qkv [3C, C] as bf16 bit patterns; b [3C], g_q, g_k [C] float.  Returns q, k, v as fp64
    [N, n_heads, C / n_heads]: projected, q and k normalised, NOT yet rotated."""
    x, w = bf16_to_f64(x_bits), bf16_to_f64(w_bits)
    N, C = x.shape
    if w.shape != (3 * C, C) or C % n_heads:
        raise ValueError("w_qkv must be [3C, C] and C a multiple of n_heads")
    b = np.zeros(3 * C) if b is None else np.asarray(b, dtype=np.float64)
    g_q = np.ones(C) if g_q is None else np.asarray(g_q, dtype=np.float64)
    g_k = np.ones(C) if g_k is None else np.asarray(g_k, dtype=np.float64)
    y = x @ w.T + b[None, :]
    q = rms_norm(y[:, :C], g_q, eps)
    k = rms_norm(y[:, C:2 * C], g_k, eps)
    v = y[:, 2 * C:]
    d = C // n_heads
    return q.reshape(N, n_heads, d), k.reshape(N, n_heads, d), v.reshape(N, n_heads, d)


def rotated_operands(x_bits, w_bits, b, g_q, g_k, eps, n_heads, T, H, W, theta=10000.0, heads=None):
    """q', k' (rotated) and v per listed head: dict head -> (q' [N, d], k' [N, d], v [N, d]), fp64."""
    q, k, v = qkv_project(x_bits, w_bits, b, g_q, g_k, eps, n_heads)
    heads = range(n_heads) if heads is None else heads
    return {a: (_o.rope_rotate_f64(q[:, a], T, H, W, theta), _o.rope_rotate_f64(k[:, a], T, H, W, theta),
                np.ascontiguousarray(v[:, a])) for a in heads}


def projected_self_attention(x_bits, w_bits, b, g_q, g_k, eps, n_heads, T, H, W, theta=10000.0, rows=None,
                             heads=None) -> np.ndarray:
    """Projection, norm, rotation and exact softmax attention; fp64 [n_rows, n_heads_listed, d]."""
    ops = rotated_operands(x_bits, w_bits, b, g_q, g_k, eps, n_heads, T, H, W, theta, heads)
    return np.stack([_o.attn_core_head(qr, kr, v, rows) for qr, kr, v in ops.values()], axis=1)


def out_project(o_bits, w_o_bits, b_o) -> np.ndarray:
    """o [N, C] (the attention output, heads side by side) and w_o [C_out, C] as bf16 bit patterns, b_o [C_out]
    float or None.  Returns y = o w_o^T + b_o as fp64 [N, C_out]."""
    o, w = bf16_to_f64(o_bits), bf16_to_f64(w_o_bits)
    o = o.reshape(o.shape[0], -1)
    if w.ndim != 2 or w.shape[1] != o.shape[1]:
        raise ValueError("w_o must be [C_out, C] with C the feature count of o")
    b = np.zeros(w.shape[0]) if b_o is None else np.asarray(b_o, dtype=np.float64)
    return o @ w.T + b[None, :]


def attention_block(x_bits, w_bits, b, g_q, g_k, eps, n_heads, T, H, W, w_o_bits, b_o, theta=10000.0,
                    rows=None) -> np.ndarray:
    """The whole attention part of a block in fp64, nothing rounded between the steps: projection, norm, rotation,
    exact softmax attention over all heads, output projection.  Returns y [n_rows, C_out]."""
    o = projected_self_attention(x_bits, w_bits, b, g_q, g_k, eps, n_heads, T, H, W, theta, rows)
    w = bf16_to_f64(w_o_bits)
    bo = np.zeros(w.shape[0]) if b_o is None else np.asarray(b_o, dtype=np.float64)
    return o.reshape(o.shape[0], -1) @ w.T + bo[None, :]
