"""ctypes front end of the fp64 CPU oracle (``regenvc_oracle.c``).

TEST INFRASTRUCTURE, not product code.  All tensors cross this boundary as
numpy arrays: bf16 data as ``uint16`` bit patterns in ``[tokens, heads,
head_dim]`` order, results as ``float64``.  Nothing here touches CUDA or the
CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "regenvc_oracle.c")
_LIB = os.path.join(_HERE, "libregenvc_oracle.so")

PAIR_ADJACENT = 0
PAIR_HALF = 1

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math) if it is stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.run(
                ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
                check=True,
            )
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    L = ctypes.CDLL(_LIB)
    i32, i64, f64 = ctypes.c_int, ctypes.c_int64, ctypes.c_double
    p = ctypes.c_void_p
    L.oracle_threads.restype = i32
    L.oracle_token_position.argtypes = [i64, i32, i32, p, p, p]
    L.oracle_token_position.restype = None
    L.oracle_rope_split.argtypes = [i32, p, p, p]
    L.oracle_rope_split.restype = None
    L.oracle_rope_pair.argtypes = [i32, i32, p, p, p]
    L.oracle_rope_pair.restype = i32
    L.oracle_rope_freq.argtypes = [f64, i32, i32]
    L.oracle_rope_freq.restype = f64
    L.oracle_rope_angle.argtypes = [i64, i32, i32, i32, i32, f64]
    L.oracle_rope_angle.restype = f64
    L.oracle_rope_rotate_head.argtypes = [p, p, i32, i32, i32, i32, i32, i32, f64, i32]
    L.oracle_rope_rotate_head.restype = i32
    L.oracle_rope_rotate_f64.argtypes = [p, p, i32, i32, i32, i32, f64]
    L.oracle_rope_rotate_f64.restype = i32
    L.oracle_widen_head.argtypes = [p, p, i64, i32, i32, i32]
    L.oracle_widen_head.restype = i32
    L.oracle_attn_core_head.argtypes = [p, p, p, i64, i64, i32, p, i64, p]
    L.oracle_attn_core_head.restype = i32
    L.oracle_attn_probs_row.argtypes = [p, p, i64, i32, i64, p]
    L.oracle_attn_probs_row.restype = i32
    L.oracle_self_attn_head.argtypes = [p, p, p, i32, i32, i32, i32, i32, f64, i32, i32, p, i64, p]
    L.oracle_self_attn_head.restype = i32
    L.oracle_cross_attn_head.argtypes = [p, p, p, i64, i64, i32, i32, i32, p, i64, p]
    L.oracle_cross_attn_head.restype = i32
    L.oracle_brute_force.argtypes = [p, p, p, i32, i32, i32, i64, i32, i32, f64, i32, i32, p, p, p]
    L.oracle_brute_force.restype = i32
    _lib = L
    return L


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 tensors are passed as uint16 bit patterns")
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def threads() -> int:
    return int(_load().oracle_threads())


def token_position(n: int, H: int, W: int):
    t, y, x = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _load().oracle_token_position(n, H, W, ctypes.byref(t), ctypes.byref(y), ctypes.byref(x))
    return t.value, y.value, x.value


def rope_split(d: int):
    a, b, c = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _load().oracle_rope_split(d, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    return a.value, b.value, c.value


def rope_pair(d: int, j: int):
    a, b, c = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _check(_load().oracle_rope_pair(d, j, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)), "rope_pair")
    return a.value, b.value, c.value


def rope_freq(theta: float, i_local: int, width: int) -> float:
    return float(_load().oracle_rope_freq(theta, i_local, width))


def rope_angle(n: int, j: int, H: int, W: int, d: int, theta: float) -> float:
    return float(_load().oracle_rope_angle(n, j, H, W, d, theta))


def rope_rotate_head(x, T, H, W, head, theta=10000.0, pairing=PAIR_ADJACENT) -> np.ndarray:
    x = _u16(x)
    N, h, d = x.shape
    assert N == T * H * W
    out = np.empty((N, d), dtype=np.float64)
    _check(_load().oracle_rope_rotate_head(_ptr(x), _ptr(out), T, H, W, h, d, head, float(theta), pairing),
           "rope_rotate_head")
    return out


def rope_rotate_f64(x, T, H, W, theta=10000.0) -> np.ndarray:
    """Rotation of one head's fp64 vectors [T*H*W, d] (adjacent pairs)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    N, d = x.shape
    assert N == T * H * W
    out = np.empty_like(x)
    _check(_load().oracle_rope_rotate_f64(_ptr(x), _ptr(out), T, H, W, d, float(theta)), "rope_rotate_f64")
    return out


def _rows(rows):
    if rows is None:
        return None, 0
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    return r, int(r.shape[0])


def attn_core_head(qr, kr, v, rows=None) -> np.ndarray:
    qr = np.ascontiguousarray(qr, dtype=np.float64)
    kr = np.ascontiguousarray(kr, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    n_q, d = qr.shape
    n_kv = kr.shape[0]
    assert kr.shape == (n_kv, d) and v.shape == (n_kv, d)
    r, nr = _rows(rows)
    out = np.empty((nr if r is not None else n_q, d), dtype=np.float64)
    _check(_load().oracle_attn_core_head(_ptr(qr), _ptr(kr), _ptr(v), n_q, n_kv, d, _ptr(r), nr, _ptr(out)),
           "attn_core_head")
    return out


def attn_probs_row(qr, kr, row: int) -> np.ndarray:
    qr = np.ascontiguousarray(qr, dtype=np.float64)
    kr = np.ascontiguousarray(kr, dtype=np.float64)
    n_kv, d = kr.shape
    p = np.empty((n_kv,), dtype=np.float64)
    _check(_load().oracle_attn_probs_row(_ptr(qr), _ptr(kr), n_kv, d, row, _ptr(p)), "attn_probs_row")
    return p


def self_attn_head(q, k, v, T, H, W, head, theta=10000.0, rows=None, pairing=PAIR_ADJACENT) -> np.ndarray:
    q, k, v = _u16(q), _u16(k), _u16(v)
    N, h, d = q.shape
    assert N == T * H * W and k.shape == q.shape and v.shape == q.shape
    r, nr = _rows(rows)
    out = np.empty((nr if r is not None else N, d), dtype=np.float64)
    _check(_load().oracle_self_attn_head(_ptr(q), _ptr(k), _ptr(v), T, H, W, h, d, float(theta), pairing,
                                         head, _ptr(r), nr, _ptr(out)), "self_attn_head")
    return out


def cross_attn_head(q, k, v, head, rows=None) -> np.ndarray:
    q, k, v = _u16(q), _u16(k), _u16(v)
    n_q, h, d = q.shape
    n_kv = k.shape[0]
    assert k.shape == (n_kv, h, d) and v.shape == (n_kv, h, d)
    r, nr = _rows(rows)
    out = np.empty((nr if r is not None else n_q, d), dtype=np.float64)
    _check(_load().oracle_cross_attn_head(_ptr(q), _ptr(k), _ptr(v), n_q, n_kv, h, d, head, _ptr(r), nr,
                                          _ptr(out)), "cross_attn_head")
    return out


def self_attention(q, k, v, T, H, W, theta=10000.0, rows=None, heads=None, pairing=PAIR_ADJACENT) -> np.ndarray:
    """All (or the listed) heads; returns fp64 [n_rows, n_heads_listed, d]."""
    h = q.shape[1]
    heads = list(range(h)) if heads is None else list(heads)
    outs = [self_attn_head(q, k, v, T, H, W, a, theta, rows, pairing) for a in heads]
    return np.stack(outs, axis=1)


def cross_attention(q, k, v, rows=None, heads=None) -> np.ndarray:
    h = q.shape[1]
    heads = list(range(h)) if heads is None else list(heads)
    outs = [cross_attn_head(q, k, v, a, rows) for a in heads]
    return np.stack(outs, axis=1)


def brute_force(q, k, v, T, H, W, head, theta=10000.0, rope=True, want_matrices=False):
    q, k, v = _u16(q), _u16(k), _u16(v)
    n_q, h, d = q.shape
    n_kv = k.shape[0]
    assert n_q == T * H * W
    out = np.empty((n_q, d), dtype=np.float64)
    S = np.empty((n_q, n_kv), dtype=np.float64) if want_matrices else None
    P = np.empty((n_q, n_kv), dtype=np.float64) if want_matrices else None
    _check(_load().oracle_brute_force(_ptr(q), _ptr(k), _ptr(v), T, H, W, n_kv, h, d, float(theta),
                                      1 if rope else 0, head, _ptr(out), _ptr(S), _ptr(P)), "brute_force")
    return (out, S, P) if want_matrices else out
