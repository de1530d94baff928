"""The fused producer (QKV projection + RMS norm + rotation + operand layout) and the attention that consumes its
output, against the fp64 oracle of the same steps, through the C ABI binding."""
import numpy as np
import pytest
import torch

import oracle
from oracle import qkv_oracle as qo
from paper_2607_28144_b200 import binding, synth
from parity_util import assert_parity, f64

pytestmark = pytest.mark.gpu
D = 128


def _inputs(N, h, seed, bias=True, gains=True):
    w = synth.Workload(name="t", seed=seed, T=1, H=1, W=N, n_heads=h, layers=1)
    x, wq, b, gq, gk, eps = synth.block_inputs(w)
    return x, wq, (b if bias else None), (gq if gains else None), (gk if gains else None), eps


def _run_producer(x, wq, b, gq, gk, eps, T, H, W, h, theta=10000.0):
    dev = torch.device("cuda:0")
    d = lambda t: None if t is None else t.to(dev)  # noqa: E731
    N = T * H * W
    n_pad = (N + 127) // 128 * 128
    need = binding.regenvc_prepared_bytes(N, h)
    prepared = torch.full((need + 512,), 0xEE, dtype=torch.uint8, device=dev)
    q_buf = torch.full((N * h * D + 256,), float("nan"), dtype=torch.float16, device=dev)
    q_rot = q_buf[: N * h * D].view(N, h, D)
    binding.regenvc_qkv_rope_project(d(x), d(wq), d(b), d(gq), d(gk), eps, T, H, W, h, theta, q_rot=q_rot,
                                     prepared=prepared)
    status = binding.regenvc_device_status()
    assert status == 0, binding.status_string(status)
    assert (prepared[need:] == 0xEE).all() and torch.isnan(q_buf[N * h * D:]).all(), "wrote past an output buffer"
    kp = prepared[: h * n_pad * D * 2].view(torch.float16).view(h, n_pad, D)
    vt = prepared[h * n_pad * D * 2: need].view(torch.float16).view(h, D, n_pad)
    return q_rot, prepared, kp, vt


@pytest.mark.parametrize("grid,h,bias,gains", [((1, 1, 1), 2, True, True), ((2, 3, 4), 2, False, False),
                                               ((1, 7, 19), 4, True, True), ((3, 7, 13), 2, True, False),
                                               ((2, 10, 13), 6, True, True), ((1, 5, 77), 12, True, True)])
def test_producer_outputs_match_the_oracle_operands(grid, h, bias, gains):
    """Q', K' and V't element by element: fp16 roundings of the oracle's rotated, normalised operands."""
    T, H, W = grid
    N = T * H * W
    x, wq, b, gq, gk, eps = _inputs(N, h, 600 + N + h, bias, gains)
    q_rot, _, kp, vt = _run_producer(x, wq, b, gq, gk, eps, T, H, W, h)
    nb = lambda t: None if t is None else t.double().numpy()  # noqa: E731
    ops = qo.rotated_operands(synth.bits(x), synth.bits(wq), nb(b), nb(gq), nb(gk), eps, h, T, H, W)
    for a in range(h):
        qr, kr, v = ops[a]
        # fp32 accumulation over C bf16 products, fp32 norm and rotation, one fp16 rounding
        np.testing.assert_allclose(q_rot[:, a].double().cpu().numpy(), qr, rtol=2 ** -10, atol=2e-4)
        np.testing.assert_allclose(kp[a, :N].double().cpu().numpy(), kr, rtol=2 ** -10, atol=2e-4)
        np.testing.assert_allclose(vt[a, :, :N].double().cpu().numpy(), v.T, rtol=2 ** -10, atol=2e-4)
        assert (kp[a, N:] == 0).all() and (vt[a, :, N:] == 0).all(), "padding must be zero"


@pytest.mark.parametrize("grid,h", [((2, 3, 4), 2), ((3, 7, 13), 4), ((2, 16, 20), 6), ((1, 9, 57), 12)])
def test_fused_producer_then_attention_matches_the_oracle(grid, h):
    T, H, W = grid
    N = T * H * W
    x, wq, b, gq, gk, eps = _inputs(N, h, 700 + N + h)
    q_rot, prepared, _, vt = _run_producer(x, wq, b, gq, gk, eps, T, H, W, h)
    out = torch.full((N, h, D), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    binding.regenvc_attn_forward_prepared(q_rot, prepared, N, out)
    assert binding.regenvc_device_status() == 0
    ref = qo.projected_self_attention(synth.bits(x), synth.bits(wq), b.double().numpy(), gq.double().numpy(),
                                      gk.double().numpy(), eps, h, T, H, W)
    max_v = float(vt.float().abs().max())
    assert_parity(f64(out.cpu()), ref, max_v, f"fused producer + attention {grid} h={h}")


def test_fused_path_at_the_window_size_on_sampled_rows():
    w = synth.WORKLOADS["window_480x832"]
    x, wq, b, gq, gk, eps = synth.block_inputs(w)
    q_rot, prepared, _, vt = _run_producer(x, wq, b, gq, gk, eps, w.T, w.H, w.W, w.n_heads, w.theta)
    out = torch.empty((w.n_tokens, w.n_heads, D), dtype=torch.bfloat16, device="cuda:0")
    n0 = binding.regenvc_kernel_launch_count()
    binding.regenvc_attn_forward_prepared(q_rot, prepared, w.n_tokens, out)
    assert binding.regenvc_device_status() == 0
    assert binding.regenvc_kernel_launch_count() - n0 <= 2  # attention (+ merge of the last wave): no preparation pass
    rows = synth.sample_rows(w.n_tokens, w.H, w.W, seed=w.seed, n_random=64)
    heads = [0, 5, 11]
    ref = qo.projected_self_attention(synth.bits(x), synth.bits(wq), b.double().numpy(), gq.double().numpy(),
                                      gk.double().numpy(), eps, w.n_heads, w.T, w.H, w.W, w.theta, rows=rows, heads=heads)
    got = out.cpu()[rows][:, heads].double().numpy()
    assert_parity(got, ref, float(vt.float().abs().max()), "fused path, 480x832 window")


def test_forty_heads_of_the_large_model():
    """Model dimension 5120 = 40 heads (the large-model workloads): 20 slices per token tile exchange their sums."""
    T, H, W, h = 1, 9, 30, 40
    N = T * H * W
    x, wq, b, gq, gk, eps = _inputs(N, h, 740)
    q_rot, prepared, kp, vt = _run_producer(x, wq, b, gq, gk, eps, T, H, W, h)
    ops = qo.rotated_operands(synth.bits(x), synth.bits(wq), b.double().numpy(), gq.double().numpy(),
                              gk.double().numpy(), eps, h, T, H, W, heads=[0, 17, 39])
    for a, (qr, kr, v) in ops.items():
        np.testing.assert_allclose(q_rot[:, a].double().cpu().numpy(), qr, rtol=2 ** -10, atol=2e-4)
        np.testing.assert_allclose(kp[a, :N].double().cpu().numpy(), kr, rtol=2 ** -10, atol=2e-4)
        np.testing.assert_allclose(vt[a, :, :N].double().cpu().numpy(), v.T, rtol=2 ** -10, atol=2e-4)
    # twice the same call: the sums are added in slice order, so the result does not depend on timing
    q2, _, kp2, _ = _run_producer(x, wq, b, gq, gk, eps, T, H, W, h)
    assert torch.equal(q_rot, q2) and torch.equal(kp, kp2)


def test_producer_argument_checks():
    L = binding.lib()
    x, w, q, p = 0x100000, 0x4000000, 0x8000000, 0xC000000
    f = L.regenvc_qkv_rope_project
    ok_args = dict(T=1, H=2, W=3, h=2)
    call = lambda x_=x, w_=w, q_=q, p_=p, h=2, d=128, eps=1e-6, theta=1e4, T=1: f(  # noqa: E731
        x_, w_, None, None, None, eps, q_, p_, T, 2, 3, h, d, theta, None)
    assert call(x_=None) == binding.ERR_NULL_POINTER
    assert call(p_=None) == binding.ERR_NULL_POINTER
    assert call(T=0) == binding.ERR_BAD_SHAPE
    assert call(d=64) == binding.ERR_UNSUPPORTED
    assert call(h=3) == binding.ERR_UNSUPPORTED       # odd head count
    assert call(eps=-1.0) == binding.ERR_UNSUPPORTED
    assert call(theta=0.0) == binding.ERR_UNSUPPORTED
    assert call(x_=x + 8) == binding.ERR_MISALIGNED
    assert call(p_=p + 16) == binding.ERR_MISALIGNED
    assert call(q_=x) == binding.ERR_ALIASING
    assert ok_args
