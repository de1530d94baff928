"""The allocation-free cross-attention entry point (collected last on purpose: a run that stops at the first
failure has then already run every other test).

Some callers may not let the library allocate: a real-time window loop in which a cudaMalloc would
synchronise the device and stall the other streams, or a process whose framework pool already owns the GPU's
memory.  For them regenvc_cross_attn_forward_static() keeps its operand scratch in a fixed array inside the
library.  This test calls it through the C ABI twice in a row (the second time with a shorter key sequence,
so that stale operands of the first call are still in the array) and checks each result against the
ordinary entry point and against the fp64 oracle, within the tolerance the parity tests use.  A second test
covers the entry point's own sticky status word: an out-of-range input is reported, the report clears the
word, and the next call computes normally again.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2607_28144_b200 import binding, synth
from parity_util import MAX_ERR_FACTOR, MRE_LIMIT, assert_parity

pytestmark = pytest.mark.gpu


def _call_static(L, q, k, v, out):
    stream = torch.cuda.current_stream().cuda_stream
    return L.regenvc_cross_attn_forward_static(ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(k.data_ptr()),
                                               ctypes.c_void_p(v.data_ptr()), ctypes.c_void_p(out.data_ptr()),
                                               q.shape[0], k.shape[0], q.shape[1], q.shape[2], ctypes.c_void_p(stream))


def test_static_scratch_entry_point_matches_the_allocating_one_twice_in_a_row():
    L = binding.lib()
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(9000)
    n_q, h = 700, 12
    q = synth.from_f32(rng.standard_normal((n_q, h, 128))).to(dev)
    # start-up call, as the header asks: the first call on a device looks up the array's address (and makes the
    # driver load the library's device code, which is when the GPU reserves the array)
    warm = torch.zeros((128, h, 128), dtype=torch.bfloat16, device=dev)
    assert _call_static(L, warm, warm, warm, torch.empty_like(warm)) == binding.OK
    torch.cuda.synchronize()
    for n_kv in (512, 257):  # two calls in a row; the second leaves rows of the first behind in the array
        k = synth.from_f32(rng.standard_normal((n_kv, h, 128))).to(dev)
        v = synth.from_f32(rng.standard_normal((n_kv, h, 128))).to(dev)
        ref = torch.empty_like(q)
        binding.regenvc_cross_attn_forward(q, k, v, ref)
        assert binding.regenvc_device_status() == 0
        out = torch.full_like(q, float("nan"))
        free_before = torch.cuda.mem_get_info()[0]
        assert _call_static(L, q, k, v, out) == binding.OK
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the allocation-free entry point changed free device memory"
        got, want = out.double().cpu().numpy(), ref.double().cpu().numpy()
        assert np.isfinite(got).all()
        err = np.abs(got - want)
        max_v = float(v.float().abs().max())
        assert err.max() <= MAX_ERR_FACTOR * max_v
        assert err.sum() / np.abs(want).sum() <= MRE_LIMIT
        assert binding.regenvc_static_device_status() == 0
        exact = oracle.cross_attention(synth.bits(q.cpu()), synth.bits(k.cpu()), synth.bits(v.cpu()))
        assert_parity(got, exact, max_v, f"allocation-free entry point against the oracle, {n_kv} keys")


def test_static_scratch_status_word_is_reported_and_cleared():
    """An input beyond the fp16 operand range sets the entry point's own status word; until it is read, later
    calls skip their work.  Reading it clears it, and the next call is normal again."""
    L = binding.lib()
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(9001)
    q = synth.from_f32(rng.standard_normal((300, 2, 128))).to(dev)
    k = synth.from_f32(rng.standard_normal((140, 2, 128))).to(dev)
    v = synth.from_f32(rng.standard_normal((140, 2, 128))).to(dev)
    assert binding.regenvc_static_device_status() == 0
    bad = v.clone()
    bad[2, 0, 5] = 1e6  # a value beyond the fp16 range (keys stay bf16 here and have no such limit)
    launches = binding.regenvc_kernel_launch_count()
    assert _call_static(L, q, k, bad, torch.empty_like(q)) == binding.OK
    assert binding.regenvc_kernel_launch_count() == launches + 2  # both launches are counted
    assert binding.regenvc_static_device_status() == binding.ERR_RANGE
    assert binding.regenvc_static_device_status() == 0  # cleared by the query
    assert binding.regenvc_device_status() == 0         # the ordinary entry points' word was never touched
    out = torch.full_like(q, float("nan"))
    assert _call_static(L, q, k, v, out) == binding.OK
    assert binding.regenvc_static_device_status() == 0
    exact = oracle.cross_attention(synth.bits(q.cpu()), synth.bits(k.cpu()), synth.bits(v.cpu()))
    assert_parity(out.double().cpu().numpy(), exact, float(v.float().abs().max()), "after the status was cleared")


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    L = binding.lib()
    dev = torch.device("cuda:0")
    h = 12
    n_kv = 32768 // h + 129  # n_heads * n_kv_pad just over the built-in 16 MiB
    q = torch.zeros((4, h, 128), dtype=torch.bfloat16, device=dev)
    k = torch.zeros((n_kv, h, 128), dtype=torch.bfloat16, device=dev)
    out = torch.empty_like(q)
    assert binding.regenvc_workspace_bytes(n_kv, h) - 21_299_200 > binding.STATIC_SCRATCH_BYTES
    assert _call_static(L, q, k, k, out) == binding.ERR_STATIC_LIMIT
    assert "scratch" in binding.status_string(binding.ERR_STATIC_LIMIT)
    assert _call_static(L, q, k[:256], k[:256], q) == binding.ERR_ALIASING
    with pytest.raises(binding.RegenvcError):
        binding.regenvc_cross_attn_forward_static(q, k, k, out)
