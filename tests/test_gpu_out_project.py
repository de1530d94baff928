"""The block's output projection (y = o W_o^T + b_o on the attention output as the attention calls leave it) and the
whole attention part of a block (fused producer -> attention -> output projection) against the fp64 oracle, through
the C ABI binding."""
import numpy as np
import pytest
import torch

from oracle import qkv_oracle as qo
from paper_2607_28144_b200 import binding, synth

pytestmark = pytest.mark.gpu
D = 128
DEV = "cuda:0"


def _inputs(N, h, seed, bias=True):
    w = synth.Workload(name="t", seed=seed, T=1, H=1, W=N, n_heads=h, layers=1)
    o = synth.self_inputs(w)[2]          # any bf16 [N, h, 128] tensor stands in for an attention output
    wo, bo = synth.out_proj_inputs(w)
    return o, wo, (bo if bias else None)


def _check(y, o, wo, bo, rows=None):
    """Element by element.  The kernel accumulates the C bf16 products of an output in fp32 (error at most
    C * 2^-24 of the sum of their magnitudes, 1536 * 2^-24 < 1e-4), adds the bias in fp32 and rounds once to bf16
    (relative 2^-9): |err| <= 2^-8 |ref| + 1e-4 * sum_c |o_c w_c|."""
    ob, wb = synth.bits(o), synth.bits(wo)
    if rows is not None:
        ob = ob[rows]
    ref = qo.out_project(ob, wb, None if bo is None else bo.double().numpy())
    mag = np.abs(qo.bf16_to_f64(ob).reshape(ob.shape[0], -1)) @ np.abs(qo.bf16_to_f64(wb)).T
    got = y.cpu().double().numpy()
    if rows is not None:
        got = got[rows]
    err = np.abs(got - ref)
    bound = 2.0 ** -8 * np.abs(ref) + 1e-4 * mag + 1e-30
    worst = np.unravel_index(np.argmax(err / bound), err.shape)
    assert (err <= bound).all(), f"worst at {worst}: got {got[worst]} ref {ref[worst]}"


@pytest.mark.parametrize("N,h,bias", [(1, 2, True), (128, 2, False), (300, 2, True), (257, 4, True), (1000, 6, True),
                                       (385, 12, True), (130, 40, False)])
def test_output_projection_matches_the_oracle(N, h, bias):
    o, wo, bo = _inputs(N, h, 900 + N + h, bias)
    C = h * D
    y_buf = torch.full((N * C + 256,), float("nan"), dtype=torch.bfloat16, device=DEV)
    y = y_buf[: N * C].view(N, C)
    binding.regenvc_out_project(o.to(DEV), wo.to(DEV), None if bo is None else bo.to(DEV), y=y)
    assert binding.regenvc_device_status() == 0
    assert torch.isnan(y_buf[N * C:]).all(), "wrote past y"
    _check(y, o, wo, bo)


def test_output_projection_at_the_window_size_on_sampled_rows():
    w = synth.WORKLOADS["window_480x832"]
    o = synth.self_inputs(w)[2]
    wo, bo = synth.out_proj_inputs(w)
    y = binding.regenvc_out_project(o.to(DEV), wo.to(DEV), bo.to(DEV))
    assert binding.regenvc_device_status() == 0
    rows = synth.sample_rows(w.n_tokens, w.H, w.W, w.seed, n_random=128)
    _check(y, o, wo, bo, rows=rows)
    assert torch.isfinite(y.float()).all()


def test_identity_weights_return_the_input_bits():
    """W_o = I, no bias: every output is one product with 1.0 plus zeros, exact in fp32, and the bf16 rounding of a
    bf16 value is itself."""
    N, h = 300, 2
    o, _, _ = _inputs(N, h, 77)
    eye = torch.eye(h * D, dtype=torch.bfloat16)
    y = binding.regenvc_out_project(o.to(DEV), eye.to(DEV), None)
    assert torch.equal(y.cpu().view(torch.int16), o.view(N, h * D).view(torch.int16))


@pytest.mark.parametrize("grid,h", [((2, 3, 4), 2), ((2, 10, 13), 4), ((1, 9, 57), 6)])
def test_whole_attention_block_matches_the_oracle(grid, h):
    """Fused producer -> attention on prepared operands -> output projection, against the oracle's unrounded chain.
    Two roundings separate them: the attention output to bf16 (relative 2^-9 per element, independent over the C
    terms of an output, so about 2^-9 / sqrt(3) of the output's typical size) and y to bf16, on top of the attention
    path's own tolerance; stated as sum |err| / sum |ref| <= 5e-3 and max |err| <= 2e-2 * max |ref|."""
    T, H, W = grid
    N = T * H * W
    w = synth.Workload(name="t", seed=800 + N + h, T=T, H=H, W=W, n_heads=h, layers=1)
    x, wq, b, gq, gk, eps = synth.block_inputs(w)
    wo, bo = synth.out_proj_inputs(w)
    d = lambda t: t.to(DEV)  # noqa: E731
    q_rot, prepared = binding.regenvc_qkv_rope_project(d(x), d(wq), d(b), d(gq), d(gk), eps, T, H, W, h)
    out = torch.empty((N, h, D), dtype=torch.bfloat16, device=DEV)
    binding.regenvc_attn_forward_prepared(q_rot, prepared, N, out)
    y = binding.regenvc_out_project(out, d(wo), d(bo))
    assert binding.regenvc_device_status() == 0
    ref = qo.attention_block(synth.bits(x), synth.bits(wq), b.double().numpy(), gq.double().numpy(),
                             gk.double().numpy(), eps, h, T, H, W, synth.bits(wo), bo.double().numpy())
    got = y.cpu().double().numpy()
    err = np.abs(got - ref)
    assert err.sum() / np.abs(ref).sum() <= 5e-3, err.sum() / np.abs(ref).sum()
    assert err.max() <= 2e-2 * np.abs(ref).max(), (err.max(), np.abs(ref).max())


def test_output_projection_argument_checks():
    N, h = 128, 2
    o, wo, bo = _inputs(N, h, 5)
    od, wd = o.to(DEV), wo.to(DEV)
    L = binding.lib()
    y = torch.empty((N, h * D), dtype=torch.bfloat16, device=DEV)
    assert L.regenvc_out_project(od.data_ptr(), wd.data_ptr(), None, od.data_ptr(), N, h, D, None) == binding.ERR_ALIASING
    assert L.regenvc_out_project(od.data_ptr(), wd.data_ptr(), None, y.data_ptr(), N, 3, D, None) == binding.ERR_UNSUPPORTED
    assert L.regenvc_out_project(od.data_ptr(), wd.data_ptr(), None, y.data_ptr(), N, h, 64, None) == binding.ERR_UNSUPPORTED
    assert L.regenvc_out_project(None, wd.data_ptr(), None, y.data_ptr(), N, h, D, None) == binding.ERR_NULL_POINTER
    assert L.regenvc_out_project(od.data_ptr(), wd.data_ptr(), None, y.data_ptr(), 0, h, D, None) == binding.ERR_BAD_SHAPE
    assert L.regenvc_out_project(od.data_ptr() + 2, wd.data_ptr(), None, y.data_ptr(), N - 1, h, D, None) == binding.ERR_MISALIGNED


def test_a_sustained_loop_of_the_block_chain_stays_bit_exact():
    """One and a half seconds of the whole chain at the 480x832 window shape (producer -> attention on its operands
    -> output projection, back to back, long enough to reach the power cap): every repetition must reproduce the
    first one bit for bit -- Q', K', V't, the attention output and y -- and no bounded wait may expire.  The producer
    exchanges partial row sums between thread blocks and all three kernels hand buffers over between warps on
    barriers: a hand-over that only holds on typical timing shows up here as a changed bit."""
    import time

    w = synth.WORKLOADS["window_480x832"]
    x, wq, b, gq, gk, eps = (t.to(DEV) if torch.is_tensor(t) else t for t in synth.block_inputs(w))
    wo, bo = (t.to(DEV) for t in synth.out_proj_inputs(w))
    N, h = w.n_tokens, w.n_heads

    def chain(q_rot, prepared, out, y):
        binding.regenvc_qkv_rope_project(x, wq, b, gq, gk, eps, w.T, w.H, w.W, h, w.theta, q_rot=q_rot, prepared=prepared)
        binding.regenvc_attn_forward_prepared(q_rot, prepared, N, out)
        binding.regenvc_out_project(out, wo, bo, y)

    def buffers():
        return (torch.empty((N, h, D), dtype=torch.float16, device=DEV),
                torch.zeros((binding.regenvc_prepared_bytes(N, h),), dtype=torch.uint8, device=DEV),
                torch.empty((N, h, D), dtype=torch.bfloat16, device=DEV),
                torch.empty((N, h * D), dtype=torch.bfloat16, device=DEV))

    first, again = buffers(), buffers()
    chain(*first)
    mismatches = torch.zeros((), dtype=torch.int64, device=DEV)
    t0, reps = time.time(), 0
    while time.time() - t0 < 1.5:
        for _ in range(20):
            chain(*again)
            for a, f in zip(again, first):
                mismatches += (a.view(torch.uint8) != f.view(torch.uint8)).sum()
            reps += 1
        torch.cuda.synchronize()
    assert reps >= 40
    assert int(mismatches.item()) == 0
    assert binding.regenvc_device_status() == 0
