"""Pins for the fp64 CPU oracle: everything here runs without a GPU.

Each test ties the oracle to something other than itself: closed forms,
invariants of softmax attention and of rotary embeddings, reduction to library
fp64 routines, a brute force with separate control flow, and a stored worked
example (tests/golden/worked_example_2x3x4.txt).
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2607_28144_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example_2x3x4.txt")
D = 128


def _rand_bits(rng, n, h, scale=1.0):
    return synth.bits(synth.from_f32(rng.standard_normal((n, h, D)) * scale))


def _f64(bits_arr):
    return torch.from_numpy(bits_arr.view(np.int16).copy()).view(torch.bfloat16).double().numpy()


def _golden():
    g = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            _, key, val = line.split()
            g[key] = float(val)
    return g


def _worked_inputs():
    n = np.arange(24)[:, None]
    c = np.arange(D)[None, :]
    q = (((7 * n + 3 * c + 1) % 17) - 8) / 8.0
    k = (((5 * n + 11 * c + 2) % 13) - 6) / 8.0
    v = (((3 * n + 5 * c + 3) % 19) - 9) / 8.0
    mk = lambda a: synth.bits(synth.from_f32(a[:, None, :]))
    return mk(q), mk(k), mk(v)


# ---------------------------------------------------------------- shapes (Sec. 3.9)
def test_conditioner_kv_sizes_fix_model_dim_layers_and_token_counts():
    # The paper states 94.4 MB (T5) and 47.4 MB (CLIP) of bf16 cross-attention K/V streamed to the GPU.
    # 512 and 257 tokens x model dim 1536 (12 heads x 128) x 2 B x (K and V) x 30 layers reproduce both.
    assert 512 * 12 * 128 * 2 * 2 * 30 == 94_371_840
    assert 257 * 12 * 128 * 2 * 2 * 30 == 47_370_240
    assert round(94_371_840 / 1e6, 1) == 94.4 and round(47_370_240 / 1e6, 1) == 47.4
    w = synth.WORKLOADS["window_480x832"]
    assert (w.n_heads, w.head_dim, w.layers, w.cross_kv) == (12, 128, 30, (512,))
    assert synth.WORKLOADS["clip_77f"].cross_kv == (512, 257)
    assert [synth.WORKLOADS[n].n_tokens for n in synth.WORKLOAD_ORDER] == [128, 1792, 10920, 12480, 31200]


# ---------------------------------------------------------------- RoPE geometry
def test_split_and_pair_map():
    assert oracle.rope_split(128) == (44, 42, 42)
    assert oracle.rope_pair(128, 0) == (0, 0, 44)
    assert oracle.rope_pair(128, 21) == (0, 21, 44)
    assert oracle.rope_pair(128, 22) == (1, 0, 42)
    assert oracle.rope_pair(128, 42) == (1, 20, 42)
    assert oracle.rope_pair(128, 43) == (2, 0, 42)
    assert oracle.rope_pair(128, 63) == (2, 20, 42)


def test_token_position_is_t_major_then_y_then_x():
    H, W = 3, 4
    seen = set()
    for n in range(2 * H * W):
        t, y, x = oracle.token_position(n, H, W)
        assert n == (t * H + y) * W + x and 0 <= y < H and 0 <= x < W
        seen.add((t, y, x))
    assert len(seen) == 24


def test_frequencies_closed_form_and_theta_one():
    assert oracle.rope_freq(10000.0, 0, 44) == 1.0
    assert oracle.rope_freq(10000.0, 11, 44) == pytest.approx(0.01, rel=1e-14)  # 1e4^(-1/2)
    assert oracle.rope_freq(10000.0, 21, 42) == pytest.approx(1e-4, rel=1e-14)  # 1e4^(-1)
    for i in range(21):
        assert oracle.rope_freq(1.0, i, 42) == 1.0
    # theta = 1: every angle is the axis position itself
    H, W = 5, 7
    for n in (0, 9, 34, 69):
        t, y, x = oracle.token_position(n, H, W)
        for j, pos in ((3, t), (30, y), (60, x)):
            assert oracle.rope_angle(n, j, H, W, 128, 1.0) == float(pos)


def test_golden_closed_values():
    g = _golden()
    assert oracle.rope_split(128) == (g["split_t"], g["split_y"], g["split_x"])
    assert oracle.rope_freq(1e4, 1, 44) == pytest.approx(g["omega_t_1"], rel=1e-14)
    assert oracle.rope_freq(1e4, 1, 42) == pytest.approx(g["omega_y_1"], rel=1e-14)
    assert oracle.rope_freq(1e4, 20, 42) == pytest.approx(g["omega_x_20"], rel=1e-13)
    assert oracle.token_position(23, 3, 4) == (g["pos23_t"], g["pos23_y"], g["pos23_x"])
    assert oracle.rope_angle(23, 22, 3, 4, 128, 1e4) == pytest.approx(g["angle_tok23_pair22"], rel=1e-15)
    assert oracle.rope_angle(23, 63, 3, 4, 128, 1e4) == pytest.approx(g["angle_tok23_pair63"], rel=1e-13)
    # the same values from first principles
    assert g["omega_t_1"] == pytest.approx(10000.0 ** (-2 / 44), rel=1e-14)
    assert g["angle_tok23_pair63"] == pytest.approx(3 * 10000.0 ** (-40 / 42), rel=1e-13)


def test_rotation_is_orthogonal_identity_at_origin_and_additive():
    rng = np.random.default_rng(1)
    T, H, W = 3, 4, 5
    x = _rand_bits(rng, T * H * W, 2)
    xr = oracle.rope_rotate_head(x, T, H, W, head=1)
    xf = _f64(x)[:, 1, :]
    np.testing.assert_allclose(np.linalg.norm(xr, axis=1), np.linalg.norm(xf, axis=1), rtol=1e-14)
    np.testing.assert_array_equal(xr[0], xf[0])  # token 0 sits at the origin: R(0,0,0) = I
    # pair norms are preserved pair by pair
    np.testing.assert_allclose(xr[:, 0::2] ** 2 + xr[:, 1::2] ** 2, xf[:, 0::2] ** 2 + xf[:, 1::2] ** 2,
                               rtol=1e-13, atol=1e-15)
    # R(p) R(p') = R(p + p'): rotating the vector of token a placed at token b's position twice
    a = np.repeat(x[7:8], T * H * W, axis=0)  # same vector at every position
    ar = oracle.rope_rotate_head(a, T, H, W, head=0)
    # position (1,1,1) then again (1,1,1) equals position (2,2,2)
    n111, n222 = (1 * H + 1) * W + 1, (2 * H + 2) * W + 2
    once = ar[n111]
    z0 = _f64(a)[0, 0, 0::2] + 1j * _f64(a)[0, 0, 1::2]
    rot = (once[0::2] + 1j * once[1::2]) / z0
    twice = z0 * rot * rot
    np.testing.assert_allclose(ar[n222][0::2], twice.real, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(ar[n222][1::2], twice.imag, rtol=1e-12, atol=1e-14)


def test_rope_relativity_scores_depend_only_on_offset():
    rng = np.random.default_rng(2)
    T, H, W = 4, 5, 6
    N = T * H * W
    a = np.repeat(_rand_bits(rng, 1, 1), N, axis=0)
    b = np.repeat(_rand_bits(rng, 1, 1), N, axis=0)
    ar = oracle.rope_rotate_head(a, T, H, W, 0)
    br = oracle.rope_rotate_head(b, T, H, W, 0)
    idx = lambda t, y, x: (t * H + y) * W + x
    for (dt, dy, dx) in [(0, 0, 1), (1, 0, 0), (0, 2, 0), (1, 2, 3), (2, 1, 4)]:
        vals = []
        for t0 in range(T - dt):
            for y0 in range(H - dy):
                for x0 in range(W - dx):
                    vals.append(ar[idx(t0 + dt, y0 + dy, x0 + dx)] @ br[idx(t0, y0, x0)])
        assert len(vals) > 1
        np.testing.assert_allclose(vals, vals[0], rtol=0, atol=1e-11)
    # and it does depend on the offset
    assert abs(ar[idx(1, 0, 0)] @ br[0] - ar[idx(0, 0, 1)] @ br[0]) > 1e-3


def test_single_axis_grid_reduces_to_textbook_1d_rope():
    rng = np.random.default_rng(3)
    W = 9
    x = _rand_bits(rng, W, 1)
    xr = oracle.rope_rotate_head(x, 1, 1, W, 0)
    xf = _f64(x)[:, 0, :]
    np.testing.assert_array_equal(xr[:, :86], xf[:, :86])  # t and y blocks untouched
    # textbook 1-D RoPE of width 42 on the last 42 dims
    i = np.arange(21)
    ang = np.arange(W)[:, None] * (10000.0 ** (-2.0 * i / 42.0))[None, :]
    z = (xf[:, 86::2] + 1j * xf[:, 87::2]) * np.exp(1j * ang)
    np.testing.assert_allclose(xr[:, 86::2], z.real, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(xr[:, 87::2], z.imag, rtol=1e-13, atol=1e-15)
    # likewise T only: the first 44 dims rotate with width 44, the rest stay
    xt = oracle.rope_rotate_head(x, W, 1, 1, 0)
    np.testing.assert_array_equal(xt[:, 44:], xf[:, 44:])
    i = np.arange(22)
    ang = np.arange(W)[:, None] * (10000.0 ** (-2.0 * i / 44.0))[None, :]
    z = (xf[:, 0:44:2] + 1j * xf[:, 1:44:2]) * np.exp(1j * ang)
    np.testing.assert_allclose(xt[:, 0:44:2], z.real, rtol=1e-13, atol=1e-15)
    # and H only: dims 44..85
    xy = oracle.rope_rotate_head(x, 1, W, 1, 0)
    np.testing.assert_array_equal(xy[:, :44], xf[:, :44])
    np.testing.assert_array_equal(xy[:, 86:], xf[:, 86:])
    assert np.abs(xy[1:, 44:86] - xf[1:, 44:86]).max() > 1e-2


# ---------------------------------------------------------------- softmax / attention core
def test_probability_rows_sum_to_one_and_are_non_negative():
    rng = np.random.default_rng(4)
    q = rng.standard_normal((10, D)) * 3
    k = rng.standard_normal((301, D)) * 3
    for r in range(10):
        p = oracle.attn_probs_row(q, k, r)
        assert p.min() >= 0.0 and abs(p.sum() - 1.0) < 1e-14


def test_one_and_two_key_closed_forms():
    rng = np.random.default_rng(5)
    q, k, v = _rand_bits(rng, 1, 1), _rand_bits(rng, 1, 1), _rand_bits(rng, 1, 1)
    np.testing.assert_array_equal(oracle.self_attn_head(q, k, v, 1, 1, 1, 0), _f64(v)[:, 0])
    q = rng.standard_normal((2, D)); k = rng.standard_normal((2, D)); v = rng.standard_normal((2, D))
    o = oracle.attn_core_head(q, k, v)
    s = (q @ k.T) / math.sqrt(D)
    sig = 1.0 / (1.0 + math.exp(-(s[0, 0] - s[0, 1])))
    np.testing.assert_allclose(o[0], sig * v[0] + (1 - sig) * v[1], rtol=1e-13, atol=1e-15)


def test_zero_queries_or_keys_give_column_mean_of_v():
    rng = np.random.default_rng(6)
    T, H, W, h = 2, 5, 7, 3
    N = T * H * W
    q, k, v = _rand_bits(rng, N, h), _rand_bits(rng, N, h), _rand_bits(rng, N, h)
    zero = np.zeros_like(q)
    mean = _f64(v).mean(axis=0)
    for qq, kk in ((zero, k), (q, zero)):
        o = oracle.self_attention(qq, kk, v, T, H, W)
        np.testing.assert_allclose(o, np.broadcast_to(mean, o.shape), rtol=0, atol=1e-14)
    # identical keys (cross path, no rotation) -> mean of V
    kc = np.repeat(k[:1], 33, axis=0)
    vc = _rand_bits(rng, 33, h)
    o = oracle.cross_attention(q, kc, vc)
    np.testing.assert_allclose(o, np.broadcast_to(_f64(vc).mean(axis=0), o.shape), rtol=0, atol=1e-14)


def test_constant_v_linearity_and_convex_hull():
    rng = np.random.default_rng(7)
    T, H, W, h = 1, 6, 9, 2
    N = T * H * W
    q, k = _rand_bits(rng, N, h, 2.0), _rand_bits(rng, N, h, 2.0)
    crow = synth.from_f32(rng.standard_normal((1, h, D)))
    vconst = synth.bits(crow.expand(N, h, D).contiguous())
    o = oracle.self_attention(q, k, vconst, T, H, W)
    np.testing.assert_allclose(o, np.broadcast_to(_f64(vconst)[0], o.shape), rtol=0, atol=1e-14)
    # linearity in V with exactly representable combinations
    v1 = synth.from_f32(np.round(rng.standard_normal((N, h, D)) * 4) / 4)
    v2 = synth.from_f32(np.round(rng.standard_normal((N, h, D)) * 4) / 4)
    v3 = (v1.float() * 2 + v2.float()).to(torch.bfloat16)
    assert torch.equal(v3.float(), v1.float() * 2 + v2.float())
    o1 = oracle.self_attention(q, k, synth.bits(v1), T, H, W)
    o2 = oracle.self_attention(q, k, synth.bits(v2), T, H, W)
    o3 = oracle.self_attention(q, k, synth.bits(v3), T, H, W)
    np.testing.assert_allclose(o3, 2 * o1 + o2, rtol=0, atol=1e-13)
    vf = _f64(synth.bits(v1))
    assert (o1 <= vf.max(axis=0) + 1e-14).all() and (o1 >= vf.min(axis=0) - 1e-14).all()


def test_permuting_key_value_pairs_leaves_output_unchanged():
    rng = np.random.default_rng(8)
    n_q, n_kv, h = 17, 75, 2
    q, k, v = _rand_bits(rng, n_q, h), _rand_bits(rng, n_kv, h), _rand_bits(rng, n_kv, h)
    perm = rng.permutation(n_kv)
    o1 = oracle.cross_attention(q, k, v)
    o2 = oracle.cross_attention(q, k[perm], v[perm])
    np.testing.assert_allclose(o1, o2, rtol=0, atol=1e-14)
    # after rotation (self path): permute rotated keys together with values
    T, H, W = 2, 3, 5
    N = T * H * W
    q, k, v = _rand_bits(rng, N, 1), _rand_bits(rng, N, 1), _rand_bits(rng, N, 1)
    qr, kr = oracle.rope_rotate_head(q, T, H, W, 0), oracle.rope_rotate_head(k, T, H, W, 0)
    vf = _f64(v)[:, 0]
    perm = rng.permutation(N)
    np.testing.assert_allclose(oracle.attn_core_head(qr, kr, vf), oracle.attn_core_head(qr, kr[perm], vf[perm]),
                               rtol=0, atol=1e-14)
    np.testing.assert_allclose(oracle.attn_core_head(qr, kr, vf), oracle.self_attn_head(q, k, v, T, H, W, 0),
                               rtol=0, atol=0)


def test_dominating_key_gives_that_value_row():
    rng = np.random.default_rng(9)
    q = rng.standard_normal((4, D)); k = rng.standard_normal((50, D)); v = rng.standard_normal((50, D))
    k[13] = q[2] * 40.0
    o = oracle.attn_core_head(q, k, v)
    np.testing.assert_allclose(o[2], v[13], rtol=0, atol=1e-12)


@pytest.mark.parametrize("b", [2.0, 12.0, 23.0])
def test_one_key_above_a_flat_tail_closed_form(b):
    """q = 8 e_0; one key b e_0 with value +1, all 1999 others zero keys with value -1: the score gap is
    8 b / sqrt(128) nats, the tail's weight t = 1999 exp(-gap), and every output element (1 - t) / (1 + t)."""
    n_q, n_kv = 3, 2000
    q = np.zeros((n_q, 1, 128), dtype=np.float32)
    k = np.zeros((n_kv, 1, 128), dtype=np.float32)
    v = -np.ones((n_kv, 1, 128), dtype=np.float32)
    q[:, 0, 0] = 8.0
    k[1234, 0, 0] = b
    v[1234] = 1.0
    out = oracle.cross_attention(synth.bits(synth.from_f32(q)), synth.bits(synth.from_f32(k)), synth.bits(synth.from_f32(v)))
    t = (n_kv - 1) * math.exp(-8.0 * b / math.sqrt(128.0))
    np.testing.assert_allclose(out, (1.0 - t) / (1.0 + t), rtol=1e-12, atol=1e-15)


def test_core_equals_library_fp64_sdpa():
    rng = np.random.default_rng(10)
    q = rng.standard_normal((37, D)) * 1.5; k = rng.standard_normal((203, D)) * 1.5
    v = rng.standard_normal((203, D))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None, None], torch.from_numpy(k)[None, None], torch.from_numpy(v)[None, None])[0, 0]
    np.testing.assert_allclose(oracle.attn_core_head(q, k, v), ref.numpy(), rtol=1e-12, atol=1e-14)
    rows = [36, 0, 5, 5]
    np.testing.assert_allclose(oracle.attn_core_head(q, k, v, rows=rows), ref.numpy()[rows], rtol=1e-12, atol=1e-14)


def _torch_self_attention(q, k, v, T, H, W, theta=1e4):
    """Library formulation: complex rotation via torch.polar + fp64 SDPA."""
    qf, kf, vf = (torch.from_numpy(_f64(a)) for a in (q, k, v))
    N, h, d = qf.shape
    n = torch.arange(N)
    pos = torch.stack([n // (H * W), (n // W) % H, n % W], 1).double()
    widths = [d - 4 * (d // 6), 2 * (d // 6), 2 * (d // 6)]
    ang = torch.cat([pos[:, a:a + 1] * theta ** (-torch.arange(0, w, 2).double() / w)[None, :]
                     for a, w in enumerate(widths)], 1)  # [N, d/2]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]
    rq = torch.view_as_real(torch.view_as_complex(qf.reshape(N, h, d // 2, 2).contiguous()) * rot).reshape(N, h, d)
    rk = torch.view_as_real(torch.view_as_complex(kf.reshape(N, h, d // 2, 2).contiguous()) * rot).reshape(N, h, d)
    o = torch.nn.functional.scaled_dot_product_attention(rq.permute(1, 0, 2)[None], rk.permute(1, 0, 2)[None],
                                                         vf.permute(1, 0, 2)[None])[0]
    return o.permute(1, 0, 2).numpy(), rq.numpy()


@pytest.mark.parametrize("grid,h", [((1, 1, 1), 1), ((1, 1, 2), 1), ((2, 1, 1), 2), ((1, 3, 1), 1),
                                    ((2, 3, 4), 2), ((3, 5, 7), 3), ((2, 8, 8), 2)])
def test_full_path_against_brute_force_and_library_formulation(grid, h):
    T, H, W = grid
    rng = np.random.default_rng(100 + T * H * W)
    N = T * H * W
    q, k, v = _rand_bits(rng, N, h), _rand_bits(rng, N, h), _rand_bits(rng, N, h)
    o = oracle.self_attention(q, k, v, T, H, W)
    lib, _ = _torch_self_attention(q, k, v, T, H, W)
    np.testing.assert_allclose(o, lib, rtol=1e-11, atol=1e-13)
    for a in range(h):
        bf, S, P = oracle.brute_force(q, k, v, T, H, W, a, want_matrices=True)
        np.testing.assert_allclose(o[:, a], bf, rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(P.sum(axis=1), 1.0, rtol=0, atol=1e-14)
        assert np.allclose(S, S) and P.min() >= 0
    # cross form
    kc, vc = _rand_bits(rng, 7, h), _rand_bits(rng, 7, h)
    oc = oracle.cross_attention(q, kc, vc)
    for a in range(h):
        np.testing.assert_allclose(oc[:, a], oracle.brute_force(q, kc, vc, T, H, W, a, rope=False),
                                   rtol=1e-11, atol=1e-13)


def test_heads_are_independent_and_row_subsets_match():
    rng = np.random.default_rng(11)
    T, H, W, h = 2, 4, 5, 4
    N = T * H * W
    q, k, v = _rand_bits(rng, N, h), _rand_bits(rng, N, h), _rand_bits(rng, N, h)
    full = oracle.self_attention(q, k, v, T, H, W)
    # changing other heads' data does not change head 2
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    for arr in (q2, k2, v2):
        arr[:, [0, 1, 3], :] = _rand_bits(rng, N, 3)
    np.testing.assert_array_equal(oracle.self_attn_head(q2, k2, v2, T, H, W, 2), full[:, 2])
    # a two-head sub-tensor gives the same as heads 1..2 of the full call
    sub = oracle.self_attention(np.ascontiguousarray(q[:, 1:3]), np.ascontiguousarray(k[:, 1:3]),
                                np.ascontiguousarray(v[:, 1:3]), T, H, W)
    np.testing.assert_array_equal(sub, full[:, 1:3])
    rows = [0, 39, 17, 17, 3]
    np.testing.assert_array_equal(oracle.self_attention(q, k, v, T, H, W, rows=rows), full[rows])


def test_worked_example_values():
    g = _golden()
    q, k, v = _worked_inputs()
    T, H, W = 2, 3, 4
    qr = oracle.rope_rotate_head(q, T, H, W, 0)
    kr = oracle.rope_rotate_head(k, T, H, W, 0)
    for c in (0, 1, 2, 3, 44, 45, 46, 47):
        assert qr[23, c] == pytest.approx(g[f"qrot_23_{c}"], rel=1e-12, abs=1e-14)
    S = (qr @ kr.T) / math.sqrt(D)
    for (a, b) in ((0, 0), (0, 1), (5, 17), (23, 0)):
        assert S[a, b] == pytest.approx(g[f"S_{a}_{b}"], rel=1e-11, abs=1e-14)
    p5 = oracle.attn_probs_row(qr, kr, 5)
    assert int(p5.argmax()) == int(g["row5_argmax"]) and p5.max() == pytest.approx(g["row5_pmax"], rel=1e-12)
    o = oracle.self_attn_head(q, k, v, T, H, W, 0)
    for (r, c) in ((0, 0), (0, 1), (0, 2), (5, 0), (5, 1), (5, 2), (23, 125), (23, 126), (23, 127)):
        assert o[r, c] == pytest.approx(g[f"O_{r}_{c}"], rel=1e-11, abs=1e-14)
    assert o.sum() == pytest.approx(g["O_sum"], rel=1e-11)
    assert np.abs(o).sum() == pytest.approx(g["O_abs_sum"], rel=1e-12)
    oc = oracle.cross_attn_head(q, k[:7], v[:7], 0)
    for c in range(3):
        assert oc[0, c] == pytest.approx(g[f"X_O_0_{c}"], rel=1e-11, abs=1e-14)
    assert oc.sum() == pytest.approx(g["X_O_sum"], rel=1e-11)
    # the half-split pairing is a different function of the same inputs (a mix-up cannot hide in a tolerance)
    oh = oracle.self_attn_head(q, k, v, T, H, W, 0, pairing=oracle.PAIR_HALF)
    for c in range(3):
        assert oh[5, c] == pytest.approx(g[f"half_O_5_{c}"], rel=1e-11, abs=1e-14)
    assert oh.sum() == pytest.approx(g["half_O_sum"], rel=1e-11)
    assert abs(oh.sum() - o.sum()) > 1e-2


def test_bad_arguments_are_rejected():
    q = np.zeros((4, 1, D), dtype=np.uint16)
    with pytest.raises(RuntimeError):
        oracle.self_attn_head(q, q, q, 2, 2, 1, 0, theta=-1.0)
    with pytest.raises(RuntimeError):
        oracle.attn_core_head(np.zeros((2, D)), np.zeros((2, D)), np.zeros((2, D)), rows=[5])
    with pytest.raises(TypeError):
        oracle.self_attn_head(q.astype(np.float32), q, q, 2, 2, 1, 0)
