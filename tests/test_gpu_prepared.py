"""Attention on operands prepared ahead of the call: the conditioning keys/values rewritten once and reused
(Sec. 3.9), and the entry point a fused producer feeds (rotated fp16 queries, K', V't).  Everything is checked
against the fp64 oracle through the C ABI binding."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_28144_b200 import binding, synth
from parity_util import assert_parity, f64, run_gpu_cross

pytestmark = pytest.mark.gpu
D = 128


def _rand(rng, n, h, scale=1.0):
    return synth.from_f32(rng.standard_normal((n, h, D)) * scale)


@pytest.mark.parametrize("n_q,n_kv,h", [(1, 1, 1), (200, 7, 2), (700, 257, 3), (513, 512, 12), (300, 769, 2)])
def test_prepared_cross_attention_matches_the_oracle_and_the_one_call_form(n_q, n_kv, h):
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(7000 + n_q + n_kv)
    q, k, v = _rand(rng, n_q, h, 1.3), _rand(rng, n_kv, h, 1.3), _rand(rng, n_kv, h)
    n_pad = (n_kv + 127) // 128 * 128
    assert binding.regenvc_prepared_bytes(n_kv, h) == 2 * h * n_pad * D * 2
    prepared = torch.full((binding.regenvc_prepared_bytes(n_kv, h) + 512,), 0xFF, dtype=torch.uint8, device=dev)
    binding.regenvc_cross_kv_prepare(k.to(dev), v.to(dev), prepared)
    torch.cuda.synchronize()
    assert (prepared[-512:] == 0xFF).all(), "the preparation pass wrote past its buffer"
    # layout: K' keeps the bf16 bits of k, V't is v transposed in fp16, padding zero
    kp = prepared[: h * n_pad * D * 2].view(torch.bfloat16).view(h, n_pad, D).cpu()
    vt = prepared[h * n_pad * D * 2: 2 * h * n_pad * D * 2].view(torch.float16).view(h, D, n_pad).cpu()
    assert torch.equal(kp[:, :n_kv].view(torch.int16), k.permute(1, 0, 2).contiguous().view(torch.int16))
    assert (kp[:, n_kv:].float() == 0).all() and (vt[:, :, n_kv:].float() == 0).all()
    # (bf16 -> fp16 is exact except below 2^-14, where fp16 is subnormal: absolute error at most 2^-25)
    np.testing.assert_allclose(vt[:, :, :n_kv].double().numpy(), f64(v).transpose(1, 2, 0), rtol=0, atol=2.0 ** -25)
    # two calls on the same prepared operands (nothing may be consumed by a call)
    qd = q.to(dev)
    outs = []
    for _ in range(2):
        out = torch.full((n_q, h, D), float("nan"), dtype=torch.bfloat16, device=dev)
        binding.regenvc_cross_attn_forward_prepared(qd, prepared, n_kv, out)
        assert binding.regenvc_device_status() == 0
        outs.append(out.cpu())
    assert torch.equal(outs[0], outs[1])
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    assert_parity(f64(outs[0]), ref, float(v.float().abs().max()), f"prepared cross {n_q}x{n_kv}")
    assert torch.equal(outs[0], run_gpu_cross(q, k, v))  # the one-call form runs the same two kernels


def test_prepared_cross_attention_at_the_window_size_uses_one_launch_per_call():
    w = synth.WORKLOADS["window_480x832"]
    dev = torch.device("cuda:0")
    q, _, _ = synth.self_inputs(w)
    kc, vc = synth.cross_inputs(w, 512)
    prepared = binding.regenvc_cross_kv_prepare(kc.to(dev), vc.to(dev))
    qd, out = q.to(dev), torch.empty_like(q, device=dev)
    binding.regenvc_cross_attn_forward_prepared(qd, prepared, 512, out)
    n0 = binding.regenvc_kernel_launch_count()
    binding.regenvc_cross_attn_forward_prepared(qd, prepared, 512, out)
    assert binding.regenvc_kernel_launch_count() - n0 == 1
    assert binding.regenvc_device_status() == 0
    rows = synth.sample_rows(w.n_tokens, w.H, w.W, seed=w.seed)
    got = out.cpu()
    for head in (0, 7, 11):
        ref = oracle.cross_attn_head(synth.bits(q), synth.bits(kc), synth.bits(vc), head, rows=rows)
        assert_parity(got[rows, head].double().numpy(), ref, float(vc.float().abs().max()), f"head {head}")


def test_prepared_argument_checks():
    import ctypes

    L = binding.lib()
    q, p, o, k = 0x100000, 0x200000, 0x300000, 0x400000
    f = L.regenvc_cross_attn_forward_prepared
    assert f(None, p, o, 4, 4, 1, 128, None) == binding.ERR_NULL_POINTER
    assert f(q, p, o, 0, 4, 1, 128, None) == binding.ERR_BAD_SHAPE
    assert f(q, p, o, 4, 4, 1, 64, None) == binding.ERR_UNSUPPORTED
    assert f(q + 8, p, o, 4, 4, 1, 128, None) == binding.ERR_MISALIGNED
    assert f(q, p + 16, o, 4, 4, 1, 128, None) == binding.ERR_MISALIGNED   # operand buffers are 256-byte aligned
    assert f(q, p, q, 4, 4, 1, 128, None) == binding.ERR_ALIASING
    assert f(q, p, p, 4, 4, 1, 128, None) == binding.ERR_ALIASING
    g = L.regenvc_cross_kv_prepare
    assert g(k, k + 0x1000, None, 4, 1, 128, None) == binding.ERR_NULL_POINTER
    assert g(k, k + 0x1000, k, 4, 1, 128, None) == binding.ERR_ALIASING
    assert g(k, k + 0x1000, p, 4, 1, 32, None) == binding.ERR_UNSUPPORTED
    assert L.regenvc_attn_forward_prepared(q, p, None, 4, 4, 1, 128, None) == binding.ERR_NULL_POINTER
    assert binding.regenvc_prepared_bytes(0, 1) == 0 and binding.regenvc_prepared_bytes(5, 1, 64) == 0


@pytest.mark.parametrize("grid,h", [((2, 3, 4), 1), ((3, 7, 13), 2), ((2, 16, 20), 4)])
def test_attention_on_producer_written_operands(grid, h):
    """regenvc_attn_forward_prepared(): the test plays the producer -- it rotates q and k in fp64 (the oracle's
    rotation), rounds them to fp16 and lays out K' and V't -- and the result must equal the oracle's attention
    on the unrounded tensors within the usual tolerance."""
    T, H, W = grid
    N = T * H * W
    n_pad = (N + 127) // 128 * 128
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(7100 + N)
    q, k, v = _rand(rng, N, h), _rand(rng, N, h), _rand(rng, N, h)
    q_rot = np.stack([oracle.rope_rotate_head(synth.bits(q), T, H, W, a) for a in range(h)], axis=1)   # [N, h, D]
    k_rot = np.stack([oracle.rope_rotate_head(synth.bits(k), T, H, W, a) for a in range(h)], axis=0)   # [h, N, D]
    kp = torch.zeros((h, n_pad, D), dtype=torch.float16)
    kp[:, :N] = torch.from_numpy(k_rot).to(torch.float16)
    vt = torch.zeros((h, D, n_pad), dtype=torch.float16)
    vt[:, :, :N] = v.permute(1, 2, 0).to(torch.float16)
    prepared = torch.cat([kp.view(torch.uint8).flatten(), vt.view(torch.uint8).flatten()]).to(dev)
    out = torch.full((N, h, D), float("nan"), dtype=torch.bfloat16, device=dev)
    binding.regenvc_attn_forward_prepared(torch.from_numpy(q_rot).to(torch.float16).to(dev), prepared, N, out)
    assert binding.regenvc_device_status() == 0
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W)
    assert_parity(f64(out.cpu()), ref, float(v.float().abs().max()), f"producer-written operands {grid}")
