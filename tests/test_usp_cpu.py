"""Host logic of the Ulysses x Ring scheme (Sec. 3.5) without a GPU: the layout arithmetic, and the per-rank driver
on gloo ranks with CPU stand-ins for the kernels (fp64 arithmetic written from the definitions, test code only),
checked against the fp64 oracle of the unsharded sequence."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_28144_b200.usp import UspLayout  # noqa: E402

D = 128


# ------------------------------------------------------------------ layout
@pytest.mark.parametrize("world,U,R,N,h", [(8, 4, 2, 10920, 12), (8, 4, 2, 12480, 40), (6, 3, 2, 1001, 6),
                                           (4, 1, 4, 77, 5), (4, 4, 1, 131, 8), (1, 1, 1, 9, 3)])
def test_layout_partitions_tokens_and_heads(world, U, R, N, h):
    L = UspLayout(world, U, R, N, h)
    shards = [L.shard(g) for g in range(world)]
    assert shards[0][0] == 0 and all(a[0] + a[1] == b[0] for a, b in zip(shards, shards[1:]))
    assert shards[-1][0] + shards[-1][1] == N
    assert max(c for _, c in shards) - min(c for _, c in shards) <= 1
    blocks = [L.block(r) for r in range(R)]
    assert blocks[0][0] == 0 and blocks[-1][0] + blocks[-1][1] == N
    for r in range(R):
        members = [L.shard(L.rank_of(u, r)) for u in range(U)]
        assert blocks[r] == (members[0][0], sum(c for _, c in members))
    heads = [L.heads(u) for u in range(U)]
    assert heads[0][0] == 0 and heads[-1][0] + heads[-1][1] == h and all(c == h // U for _, c in heads)
    assert sorted(L.rank_of(*L.coords(g)) for g in range(world)) == list(range(world))
    for g in range(world):
        u, r = L.coords(g)
        assert L.ulysses_group(g) == [r * U + i for i in range(U)] and g in L.ring_group(g)
        assert L.ring_group(g) == [i * U + u for i in range(R)]


def test_layout_of_the_paper_setting():
    L = UspLayout(8, 4, 2, 7 * 30 * 52, 12)
    assert [L.shard(g) for g in (0, 3, 4, 7)] == [(0, 1365), (4095, 1365), (5460, 1365), (9555, 1365)]
    assert L.block(0) == (0, 5460) and L.block(1) == (5460, 5460)
    assert L.heads(2) == (6, 3) and L.coords(6) == (2, 1)


@pytest.mark.parametrize("R", [1, 2, 3, 8])
def test_ring_schedule_visits_every_block_once_and_matches_the_transfers(R):
    L = UspLayout(R, 1, R, 100, 2)
    for r in range(R):
        assert sorted(L.ring_source(r, s) for s in range(R)) == list(range(R))
        assert L.ring_source(r, 0) == r
        for s in range(R - 1):
            # what r holds at step s + 1 is what its predecessor held at step s (the predecessor sent it on)
            assert L.ring_source(r, s + 1) == L.ring_source(L.ring_prev(r), s)
        assert L.ring_prev(L.ring_next(r)) == r


@pytest.mark.parametrize("kw", [dict(world=8, ulysses=4, ring=3), dict(world=4, ulysses=4, ring=1, n_heads=6),
                                dict(world=4, ulysses=2, ring=2, n_tokens=3), dict(world=32, ulysses=32, ring=1, n_heads=32)])
def test_layout_rejects_bad_settings(kw):
    base = dict(world=4, ulysses=2, ring=2, n_tokens=64, n_heads=4)
    base.update(kw)
    with pytest.raises(ValueError):
        UspLayout(**base)


# ------------------------------------------------------------------ CPU stand-ins for the kernels (test code only)
class CpuOps:
    """Tensors are float32 holding bf16 values exactly (gloo's all-to-all does not take 16-bit types)."""

    def __init__(self):
        import oracle
        self.o = oracle

    @staticmethod
    def _f64(x):
        return x.double().numpy()

    @staticmethod
    def _u16(x):
        return x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)

    @staticmethod
    def _rounded(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).float()

    def empty(self, shape, dtype, like):
        return torch.zeros(shape, dtype=dtype)

    def scatter_heads(self, x, dst, t0):
        hl = x.shape[1] // len(dst)
        for r, d in enumerate(dst):
            d[t0:t0 + x.shape[0]] = x[:, r * hl:(r + 1) * hl]

    def gather_heads(self, x, dst, token0, n_tokens, h_dst, head0):
        for d, t0, n in zip(dst, token0, n_tokens):
            assert d.shape[1] == h_dst
            d[:n, head0:head0 + x.shape[1]] = x[t0:t0 + n]

    def _rotated(self, x, T, H, W, t0, theta):
        n, h, _ = x.shape
        full = np.zeros((T * H * W, h, D), dtype=np.uint16)
        full[t0:t0 + n] = self._u16(x)
        return np.stack([self.o.rope_rotate_head(full, T, H, W, a, theta)[t0:t0 + n] for a in range(h)], axis=1)

    def partial(self, q, k, v, T, H, W, q0, kv0, theta):
        qr, kr, vv = self._rotated(q, T, H, W, q0, theta), self._rotated(k, T, H, W, kv0, theta), self._f64(v)
        s = np.einsum("nad,mad->anm", qr, kr) / np.sqrt(D) * np.log2(np.e)
        m = s.max(axis=2)
        p = np.exp2(s - m[:, :, None])
        return np.einsum("anm,mad->nad", p, vv), m.T, p.sum(axis=2).T

    def merge(self, parts, out):
        top = np.max([m for _, m, _ in parts], axis=0)
        num = sum(o * np.exp2(m - top)[:, :, None] for o, m, _ in parts)
        den = sum(l * np.exp2(m - top) for _, m, l in parts)
        out.copy_(self._rounded(num / den[:, :, None]))

    def forward(self, q, k, v, out, T, H, W, theta):
        out.copy_(self._rounded(self.o.self_attention(self._u16(q), self._u16(k), self._u16(v), T, H, W, theta)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _inputs(N, h, seed):
    from paper_2607_28144_b200 import synth
    rng = np.random.default_rng(seed)
    return [synth.from_f32(rng.standard_normal((N, h, D)) * s) for s in (1.0, 1.5, 1.0)]


def _worker(rank, world, port, U, R, grid, h, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from paper_2607_28144_b200 import usp

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        T, H, W = grid
        N = T * H * W
        layout = usp.UspLayout(world, U, R, N, h)
        t0, cnt = layout.shard(rank)
        q, k, v = (x[t0:t0 + cnt].float().contiguous() for x in _inputs(N, h, 4242))
        pg_u, pg_r = usp.make_groups(layout, rank)
        attn = usp.UspAttention(layout, rank, pg_u, pg_r, ops=CpuOps())
        o = attn(q, k, v, T, H, W)
        out[rank] = o.double().numpy()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("U,R,grid,h", [(2, 1, (1, 5, 9), 4), (1, 2, (1, 5, 9), 2), (2, 2, (2, 4, 7), 4), (1, 3, (1, 5, 8), 1)])
def test_per_rank_driver_on_gloo_ranks_equals_unsharded_attention(U, R, grid, h):
    import oracle
    from paper_2607_28144_b200 import synth

    world = U * R
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), U, R, grid, h, out), nprocs=world, join=True)
    T, H, W = grid
    N = T * H * W
    q, k, v = _inputs(N, h, 4242)
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W)
    got = np.concatenate([out[g] for g in range(world)])
    assert got.shape == ref.shape
    # the stand-ins compute in fp64, so only the final bf16 rounding separates the two
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)


def test_cuda_ops_fail_loudly_without_the_library(monkeypatch):
    from paper_2607_28144_b200 import binding, usp
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libregenvc_attn.so")
    with pytest.raises(RuntimeError):
        usp.CudaOps()
