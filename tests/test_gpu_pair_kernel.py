"""The attention kernel on pairs of thread blocks (the library picks it for long key sequences) against the oracle
at sizes the oracle finishes quickly: the calling thread's debug switch sends every call there, and the parity cases
of the other test files are run once more under it -- ragged tails, odd tile counts (a pair whose second query tile
does not exist), key-range pieces with their merge, the block-wise partial/merge pair, operands written by a producer,
and the inputs that make the optimistic run saturate so that the pair runs the item again carefully (a saturation in
one of its two thread blocks only, in one work item only, along the whole sequence).  Every case runs twice: with one
pair per work item, and on a grid of two pairs that walk over all work items (the form large calls take: the next
item's query tile prepared and its first score tiles issued while the current item finishes, finished tiles written out
by the query warps, marked items run again after the last one).  At the 480x832 window shape, where the library picks
the kernel by itself, the two kernels' outputs are compared with each other."""
import numpy as np
import pytest
import torch

import oracle
import test_gpu_blockwise
import test_gpu_parity
import test_gpu_prepared
from paper_2607_28144_b200 import binding, synth
from parity_util import assert_parity

pytestmark = pytest.mark.gpu
FORCE_PAIR, FORBID_PAIR, TWO_PAIRS_WALK, DEFAULT = 3 | 8, 3 | 16, 3 | 32, 3


@pytest.fixture(params=[FORCE_PAIR, TWO_PAIRS_WALK], ids=["pair_per_item", "two_pairs_walk"])
def pair_kernel(request):
    binding.regenvc_debug_set_phases(request.param)
    yield
    binding.regenvc_debug_set_phases(DEFAULT)


@pytest.mark.parametrize("grid,h", [((1, 1, 1), 1), ((2, 8, 8), 2), ((1, 11, 13), 3), ((3, 9, 10), 2), ((1, 16, 25), 1)])
def test_small_self_attention_shapes(pair_kernel, grid, h):
    test_gpu_parity.test_self_attention_small_shapes(grid, h)


@pytest.mark.parametrize("grid,h", [((7, 16, 16), 2), ((1, 25, 44), 3), ((2, 37, 29), 1), ((1, 40, 64), 5)])
def test_key_range_pieces_and_merge(pair_kernel, grid, h):
    test_gpu_parity.test_self_attention_with_split_key_pieces(grid, h)


@pytest.mark.parametrize("n_q,n_kv,h", [(130, 1, 1), (257, 127, 2), (300, 129, 3), (64, 769, 2), (1100, 1300, 2)])
def test_cross_attention_shapes(pair_kernel, n_q, n_kv, h):
    test_gpu_parity.test_cross_attention(n_q, n_kv, h)


@pytest.mark.parametrize("scale", [0.5, 2.0])
def test_score_range(pair_kernel, scale):
    test_gpu_parity.test_self_attention_score_range(scale)


def test_closed_forms(pair_kernel):
    test_gpu_parity.test_zero_queries_give_column_mean_everywhere()
    test_gpu_parity.test_constant_value_rows_come_back_exactly()
    test_gpu_parity.test_position_probe_values()
    test_gpu_parity.test_dominating_key_and_large_scores()


@pytest.mark.parametrize("growth", [3.0, 12.0, 40.0])
def test_second_pass_along_the_whole_sequence(pair_kernel, growth):
    test_gpu_parity.test_scores_that_grow_along_the_sequence_force_reference_updates(growth)


@pytest.mark.parametrize("key,amp", [(128 + 4, 3.5), (128 + 13, 5.0), (256 + 37, 4.0), (256 + 28, 3.5)])
def test_second_pass_after_one_jump(pair_kernel, key, amp):
    test_gpu_parity.test_one_key_far_above_the_reference_of_the_earlier_tiles(key, amp)


@pytest.mark.parametrize("key", [900, 1290])
def test_second_pass_in_one_work_item_and_one_block_of_its_pair(pair_kernel, key):
    # the saturating query rows 300..329 lie in the SECOND query tile of the item 256..511: only that thread block of
    # the pair sees the saturation, both must run the second pass
    test_gpu_parity.test_a_saturation_in_one_work_item_only(key)


def test_saturations_in_several_work_items_far_apart(pair_kernel):
    """Nine work items per head and two heads, eleven key tiles.  Query rows of items 1, 4 and 8 of head 0 and of
    item 6 of head 1 each point at a late key of their own with a score about 200 log2 units above everything else:
    those four items saturate in their optimistic run and are run again carefully -- by the walking grid after its
    last item, in list order, with clean items in between that must keep their first result."""
    n_q, n_kv, h = 2200, 1300, 2
    rng = np.random.default_rng(47)
    q = rng.standard_normal((n_q, h, test_gpu_parity.D)).astype(np.float32)
    k = rng.standard_normal((n_kv, h, test_gpu_parity.D)).astype(np.float32)
    cases = [(0, 300, 700), (0, 1100, 1290), (0, 2100, 450), (1, 1600, 1000)]   # head, first query row, key
    for hd, r0, key in cases:
        sign = rng.choice([-1.0, 1.0], size=test_gpu_parity.D).astype(np.float32)
        q[r0:r0 + 20, hd] = 3.5 * sign
        k[key, hd] = 3.5 * sign
    q, k, v = synth.from_f32(q), synth.from_f32(k), test_gpu_parity._rand(rng, n_kv, h)
    gpu = test_gpu_parity.f64(test_gpu_parity.run_gpu_cross(q, k, v))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    vmax = float(v.float().abs().max())
    for hd, r0, key in cases:
        np.testing.assert_allclose(ref[r0:r0 + 20, hd], np.broadcast_to(test_gpu_parity.f64(v)[key, hd], (20, test_gpu_parity.D)),
                                   atol=1e-9)
        assert_parity(gpu[r0:r0 + 20, hd:hd + 1], ref[r0:r0 + 20, hd:hd + 1], vmax, f"saturated rows {r0}.. of head {hd}")
    assert_parity(gpu, ref, vmax, "four saturating work items of eighteen")


def test_saturations_late_in_a_long_list_of_work_items(pair_kernel):
    """140 work items of three key tiles: on the grid of two pairs each pair walks over 70 of them, so the items that
    saturate (numbers 77 and 130 of head-major order: the 39th and the 66th of their pairs) are recorded in the second
    and third word of the pair's mask and found again from there."""
    n_q, n_kv, h = 256 * 70, 300, 2
    rng = np.random.default_rng(53)
    q = rng.standard_normal((n_q, h, test_gpu_parity.D)).astype(np.float32)
    k = rng.standard_normal((n_kv, h, test_gpu_parity.D)).astype(np.float32)
    cases = [(1, 256 * 7 + 40, 290), (1, 256 * 60 + 200, 140)]   # head, first query row, key: items 70 + 7, 70 + 60
    for hd, r0, key in cases:
        sign = rng.choice([-1.0, 1.0], size=test_gpu_parity.D).astype(np.float32)   # (each case its own direction)
        q[r0:r0 + 10, hd] = 3.5 * sign
        k[key, hd] = 3.5 * sign
    q, k, v = synth.from_f32(q), synth.from_f32(k), test_gpu_parity._rand(rng, n_kv, h)
    gpu = test_gpu_parity.f64(test_gpu_parity.run_gpu_cross(q, k, v))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    vmax = float(v.float().abs().max())
    for hd, r0, key in cases:
        np.testing.assert_allclose(ref[r0:r0 + 10, hd], np.broadcast_to(test_gpu_parity.f64(v)[key, hd], (10, test_gpu_parity.D)),
                                   atol=1e-9)
        assert_parity(gpu[r0:r0 + 10, hd:hd + 1], ref[r0:r0 + 10, hd:hd + 1], vmax, f"saturated rows {r0}.. of head {hd}")
    assert_parity(gpu, ref, vmax, "two saturating work items of 140")


@pytest.mark.parametrize("n_q,n_kv,h", [(2300, 100, 3), (3000, 128, 2), (1500, 250, 4)])
def test_many_work_items_of_one_or_two_key_tiles(pair_kernel, n_q, n_kv, h):
    # items of a single key tile (and of two): the score stream runs across two item boundaries at a time
    test_gpu_parity.test_cross_attention(n_q, n_kv, h)


@pytest.mark.parametrize("case", [0, 1, 2, 3])
def test_blockwise_partials_and_merge(pair_kernel, case):
    params = [((2, 9, 14), 2, (0, 252), [0, 126, 252]), ((3, 10, 13), 3, (0, 390), [0, 100, 257, 390]),
              ((2, 16, 20), 2, (160, 480), [0, 320, 640]), ((1, 30, 40), 1, (1000, 1200), [0, 1, 129, 700, 1200])]
    test_gpu_blockwise.test_merged_blocks_equal_unsharded_attention(*params[case])


@pytest.mark.parametrize("grid,h", [((2, 3, 4), 1), ((3, 7, 13), 2), ((2, 16, 20), 4)])
def test_operands_written_by_a_producer(pair_kernel, grid, h):
    test_gpu_prepared.test_attention_on_producer_written_operands(grid, h)


def test_a_call_that_starts_with_the_error_status_set_ends_by_itself_and_the_next_one_is_normal(pair_kernel):
    """Seven work items per head, fourteen key tiles.  After a wait has expired (a warp of its own that waits on a
    barrier nothing completes) the sticky status is set: a call that starts then must give up every wait of its own
    at once, in every role of both thread blocks of every pair and at every item of the walk, end without help and
    leave the status for the caller; the call after the status has been read is bit for bit what it was before."""
    import time

    T, H, W, h = 7, 16, 16, 2
    rng = np.random.default_rng(61)
    q, k, v = (test_gpu_parity._rand(rng, T * H * W, h) for _ in range(3))
    good = test_gpu_parity.run_gpu_self(q, k, v, T, H, W)
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    out = torch.zeros_like(qd)
    binding.regenvc_debug_expire_wait(200)
    t0 = time.time()
    binding.regenvc_attn_forward(qd, kd, vd, out, T, H, W)
    assert binding.regenvc_device_status() == binding.ERR_TIMEOUT
    assert time.time() - t0 < 5.0
    assert binding.regenvc_device_status() == 0
    assert torch.equal(test_gpu_parity.run_gpu_self(q, k, v, T, H, W), good)


@pytest.mark.parametrize("h", [296, 297])
def test_as_many_work_items_as_the_pairs_lists_hold_and_one_head_more(h):
    """16384 query rows x 296 heads are 18944 work items: on 74 pairs exactly the 256 items a pair's list holds (every
    word of the mask of items to run again in use); one head more and the call is launched with one pair per item.
    Short key sequence (200 keys), so the call stays small; the kernel on pairs is forced.  Its output must equal the
    default kernel's bit for bit (same arithmetic in the same order) and the oracle's on sampled rows of two heads."""
    n_q, n_kv = 16384, 200
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(h)
    q = torch.randn((n_q, h, 128), device=dev, generator=g).to(torch.bfloat16)
    k = torch.randn((n_kv, h, 128), device=dev, generator=g).to(torch.bfloat16)
    v = torch.randn((n_kv, h, 128), device=dev, generator=g).to(torch.bfloat16)
    outs = {}
    try:
        for name, mask in (("default", DEFAULT), ("pair", FORCE_PAIR)):
            binding.regenvc_debug_set_phases(mask)
            out = torch.full_like(q, float("nan"))
            binding.regenvc_cross_attn_forward(q, k, v, out)
            assert binding.regenvc_device_status() == 0
            outs[name] = out
    finally:
        binding.regenvc_debug_set_phases(DEFAULT)
    assert torch.equal(outs["default"], outs["pair"])
    rows = torch.tensor([0, 1, 127, 128, 255, 256, 4095, 8192, 16000, 16383], device=dev)
    heads = torch.tensor([0, h - 1], device=dev)
    qs = q[rows][:, heads].cpu().contiguous()
    ks, vs = k[:, heads].cpu().contiguous(), v[:, heads].cpu().contiguous()
    ref = oracle.cross_attention(synth.bits(qs), synth.bits(ks), synth.bits(vs))
    got = outs["pair"][rows][:, heads].double().cpu().numpy()
    assert_parity(got, ref, float(vs.float().abs().max()), f"sampled rows, {h} heads")


def test_debug_switch_argument_checks():
    L = binding.lib()
    assert L.regenvc_debug_set_phases(8) == binding.ERR_BAD_SHAPE           # neither pass selected
    assert L.regenvc_debug_set_phases(3 | 8 | 16) == binding.ERR_BAD_SHAPE  # always and never
    assert L.regenvc_debug_set_phases(3 | 32 | 16) == binding.ERR_BAD_SHAPE  # the walking form of it, and never
    assert L.regenvc_debug_set_phases(64 | 3) == binding.ERR_BAD_SHAPE
    assert L.regenvc_debug_set_phases(DEFAULT) == 0


def test_the_library_picks_the_pair_kernel_at_the_window_shape_and_both_kernels_agree():
    """480x832 window, 12 heads: 516 work items of 86 key tiles.  By itself the library takes the kernel on pairs
    (its output is what test_gpu_full_size.py compares with the oracle); forced the other way the output must agree
    within two bf16 roundings of the split into key-range pieces."""
    w = synth.WORKLOADS["window_480x832"]
    q, k, v = synth.self_inputs(w)
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    outs = {}
    try:
        for name, mask in (("default", DEFAULT), ("pair", FORCE_PAIR), ("single", FORBID_PAIR)):
            binding.regenvc_debug_set_phases(mask)
            out = torch.full_like(qd, float("nan"))
            binding.regenvc_attn_forward(qd, kd, vd, out, w.T, w.H, w.W, w.theta)
            assert binding.regenvc_device_status() == 0
            outs[name] = out.float().cpu()
    finally:
        binding.regenvc_debug_set_phases(DEFAULT)
    assert torch.equal(outs["default"], outs["pair"]), "the default call did not take the kernel on pairs"
    diff = (outs["pair"] - outs["single"]).abs()
    assert torch.isfinite(diff).all()
    assert float(diff.max()) <= 2.0 ** -7 * float(v.float().abs().max())
    assert float(diff.sum() / outs["single"].abs().sum()) <= 1.5e-3
    rows = np.unique(np.concatenate([np.arange(0, 8), np.arange(w.n_tokens - 8, w.n_tokens)]))
    ref = oracle.self_attn_head(synth.bits(q), synth.bits(k), synth.bits(v), w.T, w.H, w.W, 5, w.theta, rows=rows)
    assert_parity(outs["pair"][rows, 5].double().numpy(), ref, float(v.float().abs().max()), "pair kernel, head 5")
