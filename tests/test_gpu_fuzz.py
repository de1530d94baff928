"""Seeded random shapes and value scales against the fp64 oracle: sizes drawn around the kernel's tile edges
(128-key tiles, 256-row work items, the wave boundary at which work items are cut along the keys), several
heads, inputs of different magnitude per call.  Every case is reproducible from its index."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_28144_b200 import synth
from parity_util import assert_parity, f64, hull_check, run_gpu_cross, run_gpu_self

pytestmark = pytest.mark.gpu
D = 128
EDGES = [1, 2, 63, 64, 65, 127, 128, 129, 191, 255, 256, 257, 383, 384, 385, 511, 512, 513, 640, 769, 1023, 1025]


def _draw(rng, n, h, scale):
    return synth.from_f32(rng.standard_normal((n, h, D)) * scale)


@pytest.mark.parametrize("case", range(16))
def test_cross_attention_random_shapes(case):
    rng = np.random.default_rng(31000 + case)
    n_q = int(rng.choice(EDGES)) + int(rng.integers(0, 3)) * 256
    n_kv = int(rng.choice(EDGES))
    h = int(rng.integers(1, 6))
    qs, ks, vs = rng.choice([0.25, 1.0, 3.0]), rng.choice([0.5, 1.0, 2.0]), rng.choice([1e-3, 1.0, 50.0])
    q, k, v = _draw(rng, n_q, h, qs), _draw(rng, n_kv, h, ks), _draw(rng, n_kv, h, vs)
    gpu = f64(run_gpu_cross(q, k, v))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    hull_check(gpu, f64(v))
    assert_parity(gpu, ref, float(v.float().abs().max()), f"fuzz cross #{case} {n_q}x{n_kv} h={h}")


@pytest.mark.parametrize("case", range(12))
def test_self_attention_random_grids(case):
    rng = np.random.default_rng(32000 + case)
    T, H, W = int(rng.integers(1, 5)), int(rng.integers(1, 24)), int(rng.integers(1, 24))
    h = int(rng.integers(1, 5))
    theta = float(rng.choice([100.0, 10000.0, 5e5]))
    N = T * H * W
    qs, ks = rng.choice([0.5, 1.0, 2.0]), rng.choice([0.5, 1.0, 2.0])
    q, k, v = _draw(rng, N, h, qs), _draw(rng, N, h, ks), _draw(rng, N, h, 1.0)
    gpu = f64(run_gpu_self(q, k, v, T, H, W, theta))
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W, theta)
    hull_check(gpu, f64(v))
    assert_parity(gpu, ref, float(v.float().abs().max()), f"fuzz self #{case} {T}x{H}x{W} h={h} theta={theta}")


@pytest.mark.parametrize("case", range(4))
def test_shapes_around_the_wave_boundary(case):
    """148 SMs: item counts just below, at and above one and two waves (where the last wave is cut along keys)."""
    rng = np.random.default_rng(33000 + case)
    items = [147, 148, 149, 297][case]
    h = 1 + case % 3
    pairs = -(-items // h)
    n_q = pairs * 256 - int(rng.integers(0, 200))
    n_kv = int(rng.choice([512, 640, 1100]))
    q, k, v = _draw(rng, n_q, h, 1.0), _draw(rng, n_kv, h, 1.0), _draw(rng, n_kv, h, 1.0)
    gpu = run_gpu_cross(q, k, v)
    rows = np.unique(np.concatenate([np.arange(0, min(n_q, 300)), np.arange(max(0, n_q - 300), n_q),
                                     rng.integers(0, n_q, 200)]))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v), rows=rows)
    assert_parity(f64(gpu)[rows], ref, float(v.float().abs().max()), f"wave boundary {items} items")
