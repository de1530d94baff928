"""Pins of the producer-step oracle (projection, RMS norm over all features of a token, head split, rotation,
then attention): closed forms, invariants, brute force on tiny sizes, and special cases that reduce to the
attention oracle that is pinned on its own.  No GPU."""
import math

import numpy as np
import pytest

import oracle
from oracle import qkv_oracle as qo
from paper_2607_28144_b200 import synth

D = 128


def _bits(a):
    return synth.bits(synth.from_f32(a))


def _setup(N, h, seed, w_scale=None):
    rng = np.random.default_rng(seed)
    C = h * D
    x = _bits(rng.standard_normal((N, C)))
    w = _bits(rng.standard_normal((3 * C, C)) * (w_scale if w_scale else 1.0 / math.sqrt(C)))
    b = rng.standard_normal(3 * C) * 0.1
    gq, gk = rng.uniform(0.5, 1.5, C), rng.uniform(0.5, 1.5, C)
    return x, w, b, gq, gk


def test_rms_norm_closed_values():
    y = np.array([[3.0, 4.0], [0.0, 0.0], [1.0, -1.0]])
    out = qo.rms_norm(y, np.array([2.0, 1.0]), 0.0 + 1e-300)
    np.testing.assert_allclose(out[0], [6.0 / math.sqrt(12.5), 4.0 / math.sqrt(12.5)], rtol=1e-15)
    np.testing.assert_array_equal(out[1], [0.0, 0.0])
    np.testing.assert_allclose(out[2], [2.0, -1.0], rtol=1e-15)
    # eps enters under the root, next to the MEAN (not the sum) of squares
    np.testing.assert_allclose(qo.rms_norm(y[:1], np.ones(2), 3.5), y[:1] / 4.0, rtol=1e-15)


def test_projection_against_plain_loops_on_a_tiny_case():
    """Catches a transposed weight, a wrong third of w_qkv, a bias on the wrong side of the norm and a wrong
    head split: every output element is recomputed with scalar loops."""
    N, h, d = 3, 2, 4
    C = h * d
    rng = np.random.default_rng(1)
    x = _bits(rng.integers(-4, 5, (N, C)) / 4.0)
    w = _bits(rng.integers(-4, 5, (3 * C, C)) / 8.0)
    b = rng.integers(-3, 4, 3 * C) / 4.0
    gq, gk = rng.integers(1, 4, C) / 2.0, rng.integers(1, 4, C) / 2.0
    eps = 0.25
    q, k, v = qo.qkv_project(x, w, b, gq, gk, eps, h)
    xf, wf = qo.bf16_to_f64(x), qo.bf16_to_f64(w)
    for n in range(N):
        y = [sum(xf[n, c] * wf[f, c] for c in range(C)) + b[f] for f in range(3 * C)]
        msq = sum(t * t for t in y[:C]) / C
        msk = sum(t * t for t in y[C:2 * C]) / C
        for a in range(h):
            for c in range(d):
                f = a * d + c
                assert q[n, a, c] == pytest.approx(y[f] * gq[f] / math.sqrt(msq + eps), rel=1e-13, abs=1e-15)
                assert k[n, a, c] == pytest.approx(y[C + f] * gk[f] / math.sqrt(msk + eps), rel=1e-13, abs=1e-15)
                assert v[n, a, c] == pytest.approx(y[2 * C + f], rel=1e-13, abs=1e-15)


def test_normalised_rows_have_unit_mean_square_and_ignore_the_scale_of_x():
    x, w, b, gq, gk = _setup(9, 2, 2)
    q, k, v = qo.qkv_project(x, w, None, None, None, 0.0, 2)
    np.testing.assert_allclose((q.reshape(9, -1) ** 2).mean(axis=1), 1.0, rtol=1e-13)
    np.testing.assert_allclose((k.reshape(9, -1) ** 2).mean(axis=1), 1.0, rtol=1e-13)
    x4 = _bits(qo.bf16_to_f64(x) * 4.0)  # exact in bf16
    q4, k4, v4 = qo.qkv_project(x4, w, None, None, None, 0.0, 2)
    np.testing.assert_allclose(q4, q, rtol=1e-13)
    np.testing.assert_allclose(k4, k, rtol=1e-13)
    np.testing.assert_allclose(v4, 4.0 * v, rtol=1e-13)


def test_rotation_of_fp64_vectors_agrees_with_the_pinned_bf16_rotation_and_a_closed_value():
    T, H, W = 2, 3, 4
    rng = np.random.default_rng(3)
    x = synth.from_f32(rng.standard_normal((T * H * W, 2, D)))
    for head in range(2):
        ref = oracle.rope_rotate_head(synth.bits(x), T, H, W, head)
        got = oracle.rope_rotate_f64(x[:, head].double().numpy(), T, H, W)
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-15)
    # token 23 = (t, y, x) = (1, 2, 3): the first y pair (pair 22, elements 44 and 45) turns by the angle 2.0
    e = np.zeros((24, D))
    e[23, 44] = 1.0
    r = oracle.rope_rotate_f64(e, T, H, W)
    assert r[23, 44] == pytest.approx(math.cos(2.0), abs=1e-15) and r[23, 45] == pytest.approx(math.sin(2.0), abs=1e-15)
    assert np.count_nonzero(r) == 2


def test_identity_weights_and_unit_rows_reduce_to_plain_self_attention():
    """x in {-1, +1}: every row has mean square 1, so with W_q = W_k = W_v = I, no bias, unit gains and eps = 0
    the producer step is the identity and the whole path equals self-attention with q = k = v = x."""
    T, H, W, h = 2, 3, 5, 2
    N, C = T * H * W, h * D
    rng = np.random.default_rng(4)
    x = rng.choice([-1.0, 1.0], size=(N, C))
    w = np.concatenate([np.eye(C)] * 3, axis=0)
    got = qo.projected_self_attention(_bits(x), _bits(w), None, None, None, 0.0, h, T, H, W)
    xb = _bits(x.reshape(N, h, D))
    ref = oracle.self_attention(xb, xb, xb, T, H, W)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-13)


def test_zero_query_gain_gives_the_column_mean_of_v_and_zero_weights_give_the_value_bias():
    T, H, W, h = 1, 4, 6, 1
    N, C = T * H * W, h * D
    x, w, b, gq, gk = _setup(N, h, 5)
    out = qo.projected_self_attention(x, w, b, np.zeros(C), gk, 1e-6, h, T, H, W)
    _, _, v = qo.qkv_project(x, w, b, gq, gk, 1e-6, h)
    np.testing.assert_allclose(out[:, 0], np.broadcast_to(v[:, 0].mean(axis=0), (N, D)), rtol=1e-12, atol=1e-14)
    out = qo.projected_self_attention(x, _bits(np.zeros((3 * C, C))), b, gq, gk, 1e-6, h, T, H, W)
    np.testing.assert_allclose(out[:, 0], np.broadcast_to(b[2 * C:], (N, D)), rtol=1e-12, atol=1e-14)


def test_query_gain_acts_as_a_softmax_temperature_and_rows_subset_matches():
    T, H, W, h = 2, 2, 7, 2
    N, C = T * H * W, h * D
    x, w, b, gq, gk = _setup(N, h, 6)
    ops = qo.rotated_operands(x, w, b, gq, gk, 1e-6, h, T, H, W)
    ops3 = qo.rotated_operands(x, w, b, 3.0 * gq, gk, 1e-6, h, T, H, W)
    for a in range(h):
        np.testing.assert_allclose(ops3[a][0], 3.0 * ops[a][0], rtol=1e-13)   # q' scales, k' and v do not
        np.testing.assert_allclose(ops3[a][1], ops[a][1], rtol=0, atol=0)
        p = oracle.attn_probs_row(ops[a][0], ops[a][1], 5)
        p3 = oracle.attn_probs_row(ops3[a][0], ops[a][1], 5)
        np.testing.assert_allclose(p3, p ** 3 / (p ** 3).sum(), rtol=1e-10)
    rows = [0, 5, N - 1]
    full = qo.projected_self_attention(x, w, b, gq, gk, 1e-6, h, T, H, W)
    part = qo.projected_self_attention(x, w, b, gq, gk, 1e-6, h, T, H, W, rows=rows, heads=[1])
    np.testing.assert_array_equal(part[:, 0], full[rows, 1])


def test_output_projection_against_plain_loops_and_its_special_cases():
    """Every element by scalar loops (catches a transposed weight and a bias added per token instead of per
    feature); the identity returns its input; a permutation matrix permutes features; zero weights leave the bias."""
    N, C, Co = 3, 8, 5
    rng = np.random.default_rng(7)
    o = _bits(rng.integers(-6, 7, (N, 2, C // 2)) / 4.0)      # two heads of four features, side by side
    w = _bits(rng.integers(-4, 5, (Co, C)) / 8.0)
    b = rng.integers(-3, 4, Co) / 4.0
    y = qo.out_project(o, w, b)
    of, wf = qo.bf16_to_f64(o).reshape(N, C), qo.bf16_to_f64(w)
    assert y.shape == (N, Co)
    for n in range(N):
        for f in range(Co):
            assert y[n, f] == pytest.approx(sum(of[n, c] * wf[f, c] for c in range(C)) + b[f], rel=1e-14, abs=1e-15)
    np.testing.assert_array_equal(qo.out_project(o, _bits(np.eye(C)), None), of)
    perm = rng.permutation(C)
    np.testing.assert_array_equal(qo.out_project(o, _bits(np.eye(C)[perm]), None), of[:, perm])
    np.testing.assert_array_equal(qo.out_project(o, _bits(np.zeros((Co, C))), b), np.broadcast_to(b, (N, Co)))


def test_attention_block_reduces_to_its_parts():
    """With W_o = I and no bias the block is the projected self-attention with the heads laid side by side; in
    general it is out_project applied to that result (checked with values that survive the bf16 round trip:
    one-hot W_o rows pick single features, so nothing is rounded)."""
    T, H, W, h = 1, 3, 4, 2
    N, C = T * H * W, h * D
    x, w, b, gq, gk = _setup(N, h, 8)
    att = qo.projected_self_attention(x, w, b, gq, gk, 1e-6, h, T, H, W)
    blk = qo.attention_block(x, w, b, gq, gk, 1e-6, h, T, H, W, _bits(np.eye(C)), None)
    np.testing.assert_array_equal(blk, att.reshape(N, C))
    rng = np.random.default_rng(9)
    pick = rng.integers(0, C, size=7)
    sel = np.zeros((7, C))
    sel[np.arange(7), pick] = 2.0
    bo = rng.standard_normal(7)
    rows = [0, 3, N - 1]
    blk = qo.attention_block(x, w, b, gq, gk, 1e-6, h, T, H, W, _bits(sel), bo, rows=rows)
    np.testing.assert_allclose(blk, 2.0 * att.reshape(N, C)[rows][:, pick] + bo[None, :], rtol=1e-14, atol=1e-15)
