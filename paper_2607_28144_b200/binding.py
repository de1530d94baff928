"""Thin ctypes binding of the C ABI declared in ``include/regenvc_attn.h``.

Argument marshalling only: every step of the attention path runs in the CUDA
library.  PyTorch supplies device memory and streams.  If the shared library
is missing the first call raises; there is no CPU or library fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libregenvc_attn.so")

OK, ERR_NULL_POINTER, ERR_BAD_SHAPE, ERR_UNSUPPORTED, ERR_MISALIGNED, ERR_ALIASING, ERR_CUDA, ERR_TIMEOUT, \
    ERR_WORKSPACE, ERR_RANGE, ERR_STATIC_LIMIT, ERR_INTERNAL = range(12)
STATIC_SCRATCH_BYTES = 16 << 20

EXPORTS = [
    "regenvc_attn_forward", "regenvc_cross_attn_forward", "regenvc_attn_forward_host",
    "regenvc_cross_attn_forward_host", "regenvc_workspace_bytes", "regenvc_set_workspace",
    "regenvc_device_status", "regenvc_status_string", "regenvc_last_cuda_error", "regenvc_version",
    "regenvc_kernel_launch_count", "regenvc_shutdown", "regenvc_debug_set_phases",
    "regenvc_cross_attn_forward_static", "regenvc_static_device_status", "regenvc_attn_partial",
    "regenvc_prepared_bytes", "regenvc_cross_kv_prepare", "regenvc_cross_attn_forward_prepared",
    "regenvc_attn_forward_prepared", "regenvc_qkv_rope_project", "regenvc_out_project", "regenvc_attn_merge",
    "regenvc_ulysses_scatter_heads", "regenvc_ulysses_gather_heads", "regenvc_debug_expire_wait",
]

_lib = None


class RegenvcError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"regenvc status {code}: {text}")
        self.code = code


def lib() -> ctypes.CDLL:
    """Loads the CUDA shared library (built by ``python -m paper_2607_28144_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_28144_b200.build` "
                           "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    L.regenvc_attn_forward.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, vp]
    L.regenvc_attn_forward.restype = i32
    L.regenvc_cross_attn_forward.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
    L.regenvc_cross_attn_forward.restype = i32
    L.regenvc_cross_attn_forward_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
    L.regenvc_cross_attn_forward_static.restype = i32
    L.regenvc_attn_partial.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, f32, vp]
    L.regenvc_attn_partial.restype = i32
    L.regenvc_attn_merge.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(vp), i32, vp, i32, i32, i32, vp]
    L.regenvc_attn_merge.restype = i32
    L.regenvc_ulysses_scatter_heads.argtypes = [vp, ctypes.POINTER(vp), i32, i32, i32, i32, i32, vp]
    L.regenvc_ulysses_scatter_heads.restype = i32
    L.regenvc_ulysses_gather_heads.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                               i32, i32, i32, i32, i32, vp]
    L.regenvc_ulysses_gather_heads.restype = i32
    L.regenvc_attn_forward_host.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, vp]
    L.regenvc_attn_forward_host.restype = i32
    L.regenvc_cross_attn_forward_host.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
    L.regenvc_cross_attn_forward_host.restype = i32
    L.regenvc_prepared_bytes.argtypes = [i32, i32, i32]
    L.regenvc_prepared_bytes.restype = sz
    L.regenvc_cross_kv_prepare.argtypes = [vp, vp, vp, i32, i32, i32, vp]
    L.regenvc_cross_kv_prepare.restype = i32
    L.regenvc_cross_attn_forward_prepared.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
    L.regenvc_cross_attn_forward_prepared.restype = i32
    L.regenvc_attn_forward_prepared.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
    L.regenvc_attn_forward_prepared.restype = i32
    L.regenvc_qkv_rope_project.argtypes = [vp, vp, vp, vp, vp, f32, vp, vp, i32, i32, i32, i32, i32, f32, vp]
    L.regenvc_qkv_rope_project.restype = i32
    L.regenvc_out_project.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
    L.regenvc_out_project.restype = i32
    L.regenvc_workspace_bytes.argtypes = [i32, i32, i32]
    L.regenvc_workspace_bytes.restype = sz
    L.regenvc_set_workspace.argtypes = [vp, sz]
    L.regenvc_set_workspace.restype = i32
    L.regenvc_device_status.argtypes = [vp, ctypes.POINTER(i32)]
    L.regenvc_device_status.restype = i32
    L.regenvc_static_device_status.argtypes = [vp, ctypes.POINTER(i32)]
    L.regenvc_static_device_status.restype = i32
    L.regenvc_status_string.argtypes = [i32]
    L.regenvc_status_string.restype = ctypes.c_char_p
    L.regenvc_last_cuda_error.argtypes = []
    L.regenvc_last_cuda_error.restype = ctypes.c_char_p
    L.regenvc_version.argtypes = []
    L.regenvc_version.restype = ctypes.c_char_p
    L.regenvc_kernel_launch_count.argtypes = []
    L.regenvc_kernel_launch_count.restype = ctypes.c_ulonglong
    L.regenvc_debug_expire_wait.argtypes = [i32, vp]
    L.regenvc_debug_expire_wait.restype = i32
    L.regenvc_debug_set_phases.argtypes = [i32]
    L.regenvc_debug_set_phases.restype = i32
    L.regenvc_shutdown.argtypes = []
    L.regenvc_shutdown.restype = None
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().regenvc_status_string(code).decode()


def _check(code: int):
    if code != OK:
        text = status_string(code)
        if code == ERR_CUDA:
            text += ": " + lib().regenvc_last_cuda_error().decode()
        raise RegenvcError(code, text)


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _dev_bf16(t: torch.Tensor, name: str):
    if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or t.dim() != 3:
        raise TypeError(f"{name} must be a contiguous CUDA bf16 tensor [tokens, heads, head_dim]")


def _host_bf16(t: torch.Tensor, name: str):
    if t.dtype != torch.bfloat16 or t.is_cuda or not t.is_contiguous() or t.dim() != 3:
        raise TypeError(f"{name} must be a contiguous CPU bf16 tensor [tokens, heads, head_dim]")


def regenvc_attn_forward(q, k, v, out, T: int, H: int, W: int, rope_theta: float = 10000.0, stream=None):
    """Self-attention with fused 3D RoPE on device tensors; asynchronous on ``stream``."""
    for t, nm in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
        _dev_bf16(t, nm)
    n, h, d = q.shape
    if n != T * H * W or k.shape != q.shape or v.shape != q.shape or out.shape != q.shape:
        raise ValueError("q, k, v, out must all be [T*H*W, heads, head_dim]")
    _check(lib().regenvc_attn_forward(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), T, H, W, h, d,
                                      float(rope_theta), _stream(stream)))
    return out


def regenvc_cross_attn_forward(q, k, v, out, stream=None):
    """Cross-attention of q [n_q, h, d] to k, v [n_kv, h, d] on device tensors."""
    for t, nm in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
        _dev_bf16(t, nm)
    n_q, h, d = q.shape
    n_kv = k.shape[0]
    if k.shape != (n_kv, h, d) or v.shape != k.shape or out.shape != q.shape:
        raise ValueError("shape mismatch")
    _check(lib().regenvc_cross_attn_forward(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), n_q, n_kv, h, d,
                                            _stream(stream)))
    return out


def regenvc_prepared_bytes(n_kv: int, n_heads: int, head_dim: int = 128) -> int:
    return int(lib().regenvc_prepared_bytes(n_kv, n_heads, head_dim))


def regenvc_cross_kv_prepare(k, v, prepared=None, stream=None):
    """Rewrites conditioning keys/values [n_kv, h, d] into operand form once; returns the ``prepared`` buffer
    (a CUDA uint8 tensor, allocated here with torch when not given) for regenvc_cross_attn_forward_prepared."""
    for t, nm in ((k, "k"), (v, "v")):
        _dev_bf16(t, nm)
    n_kv, h, d = k.shape
    if v.shape != k.shape:
        raise ValueError("shape mismatch")
    need = regenvc_prepared_bytes(n_kv, h, d)
    if prepared is None:
        prepared = torch.empty((need,), dtype=torch.uint8, device=k.device)
    if prepared.dtype != torch.uint8 or not prepared.is_cuda or prepared.numel() < need:
        raise TypeError(f"prepared must be a CUDA uint8 tensor of at least {need} bytes")
    _check(lib().regenvc_cross_kv_prepare(k.data_ptr(), v.data_ptr(), prepared.data_ptr(), n_kv, h, d, _stream(stream)))
    return prepared


def regenvc_cross_attn_forward_prepared(q, prepared, n_kv: int, out, stream=None):
    """Cross-attention of q [n_q, h, d] to the n_kv conditioning tokens whose operands are in ``prepared``."""
    _dev_bf16(q, "q")
    _dev_bf16(out, "out")
    n_q, h, d = q.shape
    if out.shape != q.shape:
        raise ValueError("shape mismatch")
    if prepared.dtype != torch.uint8 or not prepared.is_cuda or prepared.numel() < regenvc_prepared_bytes(n_kv, h, d):
        raise TypeError("prepared is too small for this shape")
    _check(lib().regenvc_cross_attn_forward_prepared(q.data_ptr(), prepared.data_ptr(), out.data_ptr(), n_q, n_kv, h, d,
                                                     _stream(stream)))
    return out


def regenvc_attn_forward_prepared(q_rot, prepared, n_kv: int, out, stream=None):
    """Attention on operands already in operand form: q_rot fp16 [n_q, h, d] (rotated), ``prepared`` = K' and V't."""
    if q_rot.dtype != torch.float16 or not q_rot.is_cuda or not q_rot.is_contiguous() or q_rot.dim() != 3:
        raise TypeError("q_rot must be a contiguous CUDA fp16 tensor [tokens, heads, head_dim]")
    _dev_bf16(out, "out")
    n_q, h, d = q_rot.shape
    if out.shape != q_rot.shape:
        raise ValueError("shape mismatch")
    if prepared.dtype != torch.uint8 or not prepared.is_cuda or prepared.numel() < regenvc_prepared_bytes(n_kv, h, d):
        raise TypeError("prepared is too small for this shape")
    _check(lib().regenvc_attn_forward_prepared(q_rot.data_ptr(), prepared.data_ptr(), out.data_ptr(), n_q, n_kv, h, d,
                                               _stream(stream)))
    return out


def regenvc_qkv_rope_project(x, w_qkv, b_qkv, g_q, g_k, eps: float, T: int, H: int, W: int, n_heads: int,
                             rope_theta: float = 10000.0, q_rot=None, prepared=None, stream=None):
    """QKV projection with fused RMS norm, rotation and operand layout.  x: CUDA bf16 [T*H*W, C]; w_qkv: CUDA bf16
    [3C, C]; b_qkv (fp32 [3C]), g_q, g_k (fp32 [C]) may be None.  Returns (q_rot fp16 [N, h, 128], prepared uint8),
    allocated here with torch when not given; feed them to regenvc_attn_forward_prepared."""
    if x.dtype != torch.bfloat16 or not x.is_cuda or not x.is_contiguous() or x.dim() != 2:
        raise TypeError("x must be a contiguous CUDA bf16 tensor [tokens, C]")
    n, C = x.shape
    if n != T * H * W or C != n_heads * 128:
        raise ValueError("x must be [T*H*W, n_heads * 128]")
    if w_qkv.dtype != torch.bfloat16 or not w_qkv.is_cuda or not w_qkv.is_contiguous() or tuple(w_qkv.shape) != (3 * C, C):
        raise TypeError("w_qkv must be a contiguous CUDA bf16 tensor [3C, C]")
    for t, nm, size in ((b_qkv, "b_qkv", 3 * C), (g_q, "g_q", C), (g_k, "g_k", C)):
        if t is not None and (t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or t.numel() != size):
            raise TypeError(f"{nm} must be a contiguous CUDA fp32 tensor of {size} elements (or None)")
    if q_rot is None:
        q_rot = torch.empty((n, n_heads, 128), dtype=torch.float16, device=x.device)
    need = regenvc_prepared_bytes(n, n_heads, 128)
    if prepared is None:
        prepared = torch.empty((need,), dtype=torch.uint8, device=x.device)
    if q_rot.dtype != torch.float16 or tuple(q_rot.shape) != (n, n_heads, 128) or not q_rot.is_contiguous():
        raise TypeError("q_rot must be a contiguous CUDA fp16 tensor [tokens, heads, 128]")
    if prepared.dtype != torch.uint8 or prepared.numel() < need:
        raise TypeError(f"prepared must be a CUDA uint8 tensor of at least {need} bytes")
    ptr = lambda t: None if t is None else t.data_ptr()  # noqa: E731
    _check(lib().regenvc_qkv_rope_project(x.data_ptr(), w_qkv.data_ptr(), ptr(b_qkv), ptr(g_q), ptr(g_k), float(eps),
                                          q_rot.data_ptr(), prepared.data_ptr(), T, H, W, n_heads, 128,
                                          float(rope_theta), _stream(stream)))
    return q_rot, prepared


def regenvc_out_project(attn_out, w_o, b_o, y=None, stream=None):
    """Output projection of the block: attn_out CUDA bf16 [tokens, heads, 128] (as the attention calls write it),
    w_o CUDA bf16 [C, C], b_o CUDA fp32 [C] or None.  Returns y bf16 [tokens, C] (allocated with torch if not given)."""
    _dev_bf16(attn_out, "attn_out")
    n, h, d = attn_out.shape
    C = h * d
    if w_o.dtype != torch.bfloat16 or not w_o.is_cuda or not w_o.is_contiguous() or tuple(w_o.shape) != (C, C):
        raise TypeError("w_o must be a contiguous CUDA bf16 tensor [C, C]")
    if b_o is not None and (b_o.dtype != torch.float32 or not b_o.is_cuda or not b_o.is_contiguous() or b_o.numel() != C):
        raise TypeError(f"b_o must be a contiguous CUDA fp32 tensor of {C} elements (or None)")
    if y is None:
        y = torch.empty((n, C), dtype=torch.bfloat16, device=attn_out.device)
    if y.dtype != torch.bfloat16 or not y.is_cuda or not y.is_contiguous() or tuple(y.shape) != (n, C):
        raise TypeError("y must be a contiguous CUDA bf16 tensor [tokens, C]")
    _check(lib().regenvc_out_project(attn_out.data_ptr(), w_o.data_ptr(), None if b_o is None else b_o.data_ptr(),
                                     y.data_ptr(), n, h, d, _stream(stream)))
    return y


def regenvc_cross_attn_forward_static(q, k, v, out, stream=None):
    """Cross-attention without any device allocation by the library (for callers in a real-time loop, or
    in a process whose memory pool owns the GPU): the operand scratch is a fixed 16 MiB array inside the
    library, shared by all calls on the device, so calls must not overlap on the GPU; shapes with
    n_heads * ceil(n_kv / 128) * 128 > 32768 raise ERR_STATIC_LIMIT."""
    for t, nm in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
        _dev_bf16(t, nm)
    n_q, h, d = q.shape
    n_kv = k.shape[0]
    if k.shape != (n_kv, h, d) or v.shape != k.shape or out.shape != q.shape:
        raise ValueError("shape mismatch")
    _check(lib().regenvc_cross_attn_forward_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), n_q,
                                                   n_kv, h, d, _stream(stream)))
    return out


def regenvc_attn_partial(q, k, v, o_part, ml, T: int, H: int, W: int, q_token0: int, kv_token0: int,
                         rope_theta: float = 10000.0, stream=None):
    """Unnormalised attention of the query tokens q_token0.. against the key/value block kv_token0.. of the grid.
    o_part: CUDA fp32 [n_q, h, d]; ml: CUDA fp32 [n_q, h, 2] (reference, row sum)."""
    for t, nm in ((q, "q"), (k, "k"), (v, "v")):
        _dev_bf16(t, nm)
    n_q, h, d = q.shape
    n_kv = k.shape[0]
    if k.shape != (n_kv, h, d) or v.shape != k.shape:
        raise ValueError("shape mismatch")
    if o_part.dtype != torch.float32 or tuple(o_part.shape) != (n_q, h, d) or not o_part.is_contiguous():
        raise TypeError("o_part must be a contiguous CUDA fp32 tensor [n_q, heads, head_dim]")
    if ml.dtype != torch.float32 or tuple(ml.shape) != (n_q, h, 2) or not ml.is_contiguous():
        raise TypeError("ml must be a contiguous CUDA fp32 tensor [n_q, heads, 2]")
    _check(lib().regenvc_attn_partial(q.data_ptr(), k.data_ptr(), v.data_ptr(), o_part.data_ptr(), ml.data_ptr(),
                                      T, H, W, q_token0, n_q, kv_token0, n_kv, h, d, float(rope_theta),
                                      _stream(stream)))
    return o_part, ml


def regenvc_attn_merge(o_parts, mls, out, stream=None):
    """Merges partial results of several key/value blocks (same query range) into bf16 ``out`` [n_q, h, d]."""
    _dev_bf16(out, "out")
    n_q, h, d = out.shape
    n = len(o_parts)
    if n != len(mls):
        raise ValueError("need one (m, l) tensor per partial result")
    arr_o = (ctypes.c_void_p * n)(*[t.data_ptr() for t in o_parts])
    arr_m = (ctypes.c_void_p * n)(*[t.data_ptr() for t in mls])
    _check(lib().regenvc_attn_merge(arr_o, arr_m, n, out.data_ptr(), n_q, h, d, _stream(stream)))
    return out


def _ptr(x) -> int:
    return x.data_ptr() if isinstance(x, torch.Tensor) else int(x)


def regenvc_ulysses_scatter_heads(x_local, dst, dst_token0: int, stream=None):
    """Head-group r of this GPU's tokens ``x_local`` [n_local, h, d] goes to ``dst[r]`` [group tokens, h/len(dst), d]
    at rows ``dst_token0``...  ``dst`` holds CUDA tensors or raw device addresses (a peer GPU's mapped buffer)."""
    _dev_bf16(x_local, "x_local")
    n, h, d = x_local.shape
    world = len(dst)
    arr = (ctypes.c_void_p * world)(*[_ptr(t) for t in dst])
    _check(lib().regenvc_ulysses_scatter_heads(x_local.data_ptr(), arr, world, n, int(dst_token0), h, d,
                                               _stream(stream)))


def regenvc_ulysses_gather_heads(x_heads, dst, token0, n_tokens, n_heads_dst: int, dst_head0: int, stream=None):
    """Tokens ``token0[r]``.. (``n_tokens[r]`` of them) of this GPU's heads ``x_heads`` [tokens, h_local, d] go to
    ``dst[r]`` [n_tokens[r], n_heads_dst, d] at heads ``dst_head0``...  ``dst`` as in the scatter call."""
    _dev_bf16(x_heads, "x_heads")
    _, h_loc, d = x_heads.shape
    world = len(dst)
    if len(token0) != world or len(n_tokens) != world:
        raise ValueError("need one token range per destination")
    if any(t0 < 0 or n < 0 or t0 + n > x_heads.shape[0] for t0, n in zip(token0, n_tokens)):
        raise ValueError("token range outside x_heads")
    arr = (ctypes.c_void_p * world)(*[_ptr(t) for t in dst])
    a0 = (ctypes.c_int * world)(*[int(x) for x in token0])
    an = (ctypes.c_int * world)(*[int(x) for x in n_tokens])
    _check(lib().regenvc_ulysses_gather_heads(x_heads.data_ptr(), arr, a0, an, world, h_loc, int(n_heads_dst),
                                              int(dst_head0), d, _stream(stream)))


def regenvc_attn_forward_host(q, k, v, out, T: int, H: int, W: int, rope_theta: float = 10000.0, stream=None):
    """Same operation with all four tensors in host memory (copies inside the call; returns when done)."""
    for t, nm in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
        _host_bf16(t, nm)
    n, h, d = q.shape
    if n != T * H * W or k.shape != q.shape or v.shape != q.shape or out.shape != q.shape:
        raise ValueError("q, k, v, out must all be [T*H*W, heads, head_dim]")
    _check(lib().regenvc_attn_forward_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), T, H, W, h, d,
                                           float(rope_theta), _stream(stream)))
    return out


def regenvc_cross_attn_forward_host(q, k, v, out, stream=None):
    for t, nm in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
        _host_bf16(t, nm)
    n_q, h, d = q.shape
    n_kv = k.shape[0]
    if k.shape != (n_kv, h, d) or v.shape != k.shape or out.shape != q.shape:
        raise ValueError("shape mismatch")
    _check(lib().regenvc_cross_attn_forward_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), n_q, n_kv,
                                                 h, d, _stream(stream)))
    return out


def regenvc_workspace_bytes(n_kv: int, n_heads: int, head_dim: int = 128) -> int:
    return int(lib().regenvc_workspace_bytes(n_kv, n_heads, head_dim))


def regenvc_set_workspace(buf: Optional[torch.Tensor]):
    """Use ``buf`` (a CUDA uint8 tensor the caller keeps alive) as this thread's workspace; None resets."""
    if buf is None:
        _check(lib().regenvc_set_workspace(None, 0))
    else:
        _check(lib().regenvc_set_workspace(buf.data_ptr(), buf.numel() * buf.element_size()))


def regenvc_device_status(stream=None) -> int:
    """Waits for ``stream`` and returns (then clears) the sticky device status."""
    st = ctypes.c_int(0)
    _check(lib().regenvc_device_status(_stream(stream), ctypes.byref(st)))
    return st.value


def regenvc_static_device_status(stream=None) -> int:
    """Waits for ``stream`` and returns (then clears) the status word of the allocation-free entry point."""
    st = ctypes.c_int(0)
    _check(lib().regenvc_static_device_status(_stream(stream), ctypes.byref(st)))
    return st.value


def regenvc_version() -> str:
    return lib().regenvc_version().decode()


def regenvc_kernel_launch_count() -> int:
    return int(lib().regenvc_kernel_launch_count())


def regenvc_debug_set_phases(mask: int):
    """Profiling aid: 1 = preparation pass only, 2 = attention kernel only, 3 = both (default); + 4: no persistent
    form for short key sequences; + 8 / + 16: always / never the kernel on pairs of thread blocks; + 32: always that
    kernel, on a grid of two pairs that walk over all work items."""
    _check(lib().regenvc_debug_set_phases(mask))


def regenvc_debug_expire_wait(limit_us: int = 500, stream=None):
    """Test aid: one warp waits limit_us on a barrier nothing completes; the sticky status becomes ERR_TIMEOUT."""
    _check(lib().regenvc_debug_expire_wait(int(limit_us), _stream(stream)))


def regenvc_shutdown():
    lib().regenvc_shutdown()
