"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI
binding on seeded inputs and compare with the fp64 oracle.

Tolerance (bf16 inputs, fp32 accumulation), stated once here and used by every
parity test:
    max |o_gpu - o_ref|               <= 1e-2 * max |V|
    sum |o_gpu - o_ref| / sum |o_ref| <= 2e-3        ("mean relative error")
"""
import numpy as np
import torch

import oracle
from paper_2607_28144_b200 import binding, synth

MAX_ERR_FACTOR = 1e-2
MRE_LIMIT = 2e-3
GUARD = 4096  # bf16 elements either side of the output


def _nan_bf16(n, device):
    return torch.full((n,), float("nan"), dtype=torch.bfloat16, device=device)


def run_gpu_self(q, k, v, T, H, W, theta=10000.0):
    """q, k, v: CPU bf16.  Returns the GPU result as a CPU bf16 tensor; checks guards and status."""
    dev = torch.device("cuda:0")
    n = q.numel()
    buf = _nan_bf16(n + 2 * GUARD, dev)
    out = buf[GUARD:GUARD + n].view(q.shape)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    binding.regenvc_attn_forward(qd, kd, vd, out, T, H, W, theta)
    status = binding.regenvc_device_status()
    assert status == 0, f"device status {status}: {binding.status_string(status)}"
    assert torch.isnan(buf[:GUARD]).all() and torch.isnan(buf[GUARD + n:]).all(), "guard band overwritten"
    return out.cpu()


def run_gpu_cross(q, k, v):
    dev = torch.device("cuda:0")
    n = q.numel()
    buf = _nan_bf16(n + 2 * GUARD, dev)
    out = buf[GUARD:GUARD + n].view(q.shape)
    binding.regenvc_cross_attn_forward(q.to(dev), k.to(dev), v.to(dev), out)
    status = binding.regenvc_device_status()
    assert status == 0, f"device status {status}: {binding.status_string(status)}"
    assert torch.isnan(buf[:GUARD]).all() and torch.isnan(buf[GUARD + n:]).all(), "guard band overwritten"
    return out.cpu()


def errors(gpu_rows: np.ndarray, ref_rows: np.ndarray, max_v: float):
    """gpu_rows, ref_rows: fp64 arrays of the same shape."""
    assert gpu_rows.shape == ref_rows.shape
    assert np.isfinite(gpu_rows).all(), "non-finite value in the GPU output (unwritten or overflowed element)"
    diff = np.abs(gpu_rows - ref_rows)
    denom = np.abs(ref_rows).sum()
    return {
        "max_err": float(diff.max()),
        "max_err_over_maxv": float(diff.max() / max_v) if max_v > 0 else float(diff.max()),
        "mre": float(diff.sum() / denom) if denom > 0 else float(diff.sum()),
        "l2": float(np.sqrt((diff ** 2).sum() / max((ref_rows ** 2).sum(), 1e-300))),
    }


def assert_parity(gpu_rows, ref_rows, max_v, what=""):
    e = errors(gpu_rows, ref_rows, max_v)
    if not (e["max_err"] <= MAX_ERR_FACTOR * max_v and e["mre"] <= MRE_LIMIT):
        diff = np.abs(gpu_rows - ref_rows)
        flat = diff.reshape(diff.shape[0], -1).max(axis=1)
        bad_rows = np.argsort(-flat)[:8]
        cols = diff.reshape(-1, diff.shape[-1]).max(axis=0)
        raise AssertionError(f"parity failed {what}: {e}; worst rows {bad_rows.tolist()} "
                             f"(err {flat[bad_rows].round(4).tolist()}); worst cols {np.argsort(-cols)[:8].tolist()}")
    return e


def hull_check(gpu: np.ndarray, v_f64: np.ndarray, slack=1e-2):
    """Every output lies inside the per-(head, column) range of V (attention is a convex combination)."""
    lo, hi = v_f64.min(axis=0), v_f64.max(axis=0)
    span = np.maximum(hi - lo, np.abs(hi)) * slack + 1e-6
    assert (gpu <= hi + span).all() and (gpu >= lo - span).all(), "output outside the convex hull of V"


def f64(t: torch.Tensor) -> np.ndarray:
    return t.double().numpy()
