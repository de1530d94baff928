"""Block-wise attention: partial results over key/value blocks, merged by the online-softmax rule, reproduce
unsharded attention (the paper's Sec. 3.5: its sequence parallelism changes only the order of the sums, not the
result).  Checked against the fp64 oracle of the WHOLE sequence, so a wrong rotary offset of a block, a wrong
reference or a wrong merge weight all show."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_28144_b200 import binding, synth
from parity_util import assert_parity, f64

pytestmark = pytest.mark.gpu
D = 128


def _blockwise(q, k, v, T, H, W, q_range, kv_cuts):
    dev = torch.device("cuda:0")
    q0, q1 = q_range
    qd = q[q0:q1].contiguous().to(dev)
    n_q, h = q1 - q0, q.shape[1]
    o_parts, mls = [], []
    for a, b in zip(kv_cuts[:-1], kv_cuts[1:]):
        o = torch.full((n_q, h, D), float("nan"), dtype=torch.float32, device=dev)
        ml = torch.full((n_q, h, 2), float("nan"), dtype=torch.float32, device=dev)
        binding.regenvc_attn_partial(qd, k[a:b].contiguous().to(dev), v[a:b].contiguous().to(dev), o, ml,
                                     T, H, W, q0, a)
        o_parts.append(o)
        mls.append(ml)
    out = torch.full((n_q, h, D), float("nan"), dtype=torch.bfloat16, device=dev)
    binding.regenvc_attn_merge(o_parts, mls, out)
    assert binding.regenvc_device_status() == 0
    return out.cpu(), o_parts, mls


@pytest.mark.parametrize("grid,h,q_range,cuts", [
    ((2, 9, 14), 2, (0, 252), [0, 126, 252]),            # ring of two equal halves
    ((3, 10, 13), 3, (0, 390), [0, 100, 257, 390]),      # three ragged blocks
    ((2, 16, 20), 2, (160, 480), [0, 320, 640]),         # a query shard in the middle of the sequence
    ((1, 30, 40), 1, (1000, 1200), [0, 1, 129, 700, 1200]),  # a one-token block, blocks across tile boundaries
])
def test_merged_blocks_equal_unsharded_attention(grid, h, q_range, cuts):
    T, H, W = grid
    N = T * H * W
    rng = np.random.default_rng(7000 + N + h)
    q = synth.from_f32(rng.standard_normal((N, h, D)))
    k = synth.from_f32(rng.standard_normal((N, h, D)) * 1.5)
    v = synth.from_f32(rng.standard_normal((N, h, D)))
    assert cuts[0] == 0 and cuts[-1] == N
    out, o_parts, mls = _blockwise(q, k, v, T, H, W, q_range, cuts)
    rows = np.arange(q_range[0], q_range[1])
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W, rows=rows)
    assert_parity(f64(out), ref, float(v.float().abs().max()), f"blockwise {grid} {cuts}")
    # one block covering everything is ordinary attention; the partial itself is o / l
    dev = torch.device("cuda:0")
    full = torch.empty((N, h, D), dtype=torch.bfloat16, device=dev)
    binding.regenvc_attn_forward(q.to(dev), k.to(dev), v.to(dev), full, T, H, W)
    got_vs_full = (out.float() - full[q_range[0]:q_range[1]].cpu().float()).abs().max()
    assert float(got_vs_full) <= 2 ** -7 * float(v.float().abs().max())
    for o, ml in zip(o_parts, mls):
        assert torch.isfinite(o).all() and torch.isfinite(ml).all() and (ml[..., 1] > 0).all()


def test_partial_of_a_single_block_normalises_to_attention_over_that_block():
    T, H, W, h = 1, 12, 25, 2
    N = T * H * W
    rng = np.random.default_rng(7100)
    q, k, v = (synth.from_f32(rng.standard_normal((N, h, D))) for _ in range(3))
    out, o_parts, mls = _blockwise(q, k, v, T, H, W, (0, N), [0, N])
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W)
    assert_parity(f64(out), ref, float(v.float().abs().max()), "single block")
    norm = (o_parts[0] / mls[0][..., 1:2]).cpu().double().numpy()
    np.testing.assert_allclose(norm, ref, rtol=0, atol=2e-3 * float(v.float().abs().max()))


def test_blockwise_argument_checks():
    L = binding.lib()
    a = 0x10000
    f = L.regenvc_attn_partial
    assert f(a, a + 0x10000, a + 0x20000, a + 0x30000, None, 2, 2, 2, 0, 8, 0, 8, 1, 128, 1e4, None) == binding.ERR_NULL_POINTER
    assert f(a, a + 0x10000, a + 0x20000, a + 0x30000, a + 0x50000, 2, 2, 2, 4, 8, 0, 8, 1, 128, 1e4, None) == binding.ERR_BAD_SHAPE
    assert f(a, a + 0x10000, a + 0x20000, a + 0x30000, a + 0x50000, 2, 2, 2, 0, 8, -1, 8, 1, 128, 1e4, None) == binding.ERR_BAD_SHAPE
    assert f(a, a + 0x10000, a + 0x20000, a + 0x30000, a + 0x50000, 2, 2, 2, 0, 8, 0, 8, 1, 64, 1e4, None) == binding.ERR_UNSUPPORTED
    assert f(a, a + 0x10000, a + 0x20000, a, a + 0x50000, 2, 2, 2, 0, 8, 0, 8, 1, 128, 1e4, None) == binding.ERR_ALIASING
    assert L.regenvc_attn_merge(None, None, 1, a, 8, 1, 128, None) == binding.ERR_NULL_POINTER
