"""Ulysses x Ring on one GPU: the resharding kernels against their index definition (bit-exact), and the whole
scheme, all ranks executed one after another, against the fp64 oracle of the UNSHARDED sequence (Sec. 3.5: the
parallel form changes the order of the sums, nothing else)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_28144_b200 import binding, synth, usp
from parity_util import assert_parity, f64

pytestmark = pytest.mark.gpu
D = 128
POISON = 0x7FC1  # a NaN bit pattern no input contains


def _bits(shape, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randint(0, 0x7F00, shape, generator=g, dtype=torch.int32).to(torch.int16)  # finite bf16 patterns
    return x.view(torch.bfloat16)


def _poisoned(shape, dev):
    return torch.full(shape, POISON, dtype=torch.int16, device=dev).view(torch.bfloat16)


@pytest.mark.parametrize("world,n_local,h,token0,extra", [
    (1, 5, 3, 0, 0), (2, 7, 4, 3, 2), (4, 129, 8, 0, 0), (3, 1, 6, 10, 5), (8, 33, 40, 64, 1), (16, 2, 16, 0, 0),
])
def test_scatter_heads_matches_its_definition_bitwise(world, n_local, h, token0, extra):
    dev = torch.device("cuda:0")
    x = _bits((n_local, h, D), 100 + world).to(dev)
    rows = token0 + n_local + extra
    dst = [_poisoned((rows, h // world, D), dev) for _ in range(world)]
    binding.regenvc_ulysses_scatter_heads(x, dst, token0)
    torch.cuda.synchronize()
    hl = h // world
    for r in range(world):
        got = dst[r].view(torch.int16)
        want = torch.full_like(got, POISON)
        want[token0:token0 + n_local] = x[:, r * hl:(r + 1) * hl].view(torch.int16)
        assert torch.equal(got, want), f"destination {r}"  # also: nothing outside the range was touched


@pytest.mark.parametrize("world,ranges,h_loc,h_dst,head0", [
    (1, [(0, 9)], 2, 2, 0), (2, [(0, 5), (5, 6)], 3, 6, 3), (4, [(0, 40), (40, 41), (81, 40), (121, 7)], 2, 8, 4),
    (3, [(7, 0), (0, 7), (7, 13)], 5, 40, 35), (8, [(i * 17, 17) for i in range(8)], 5, 40, 10),
])
def test_gather_heads_matches_its_definition_bitwise(world, ranges, h_loc, h_dst, head0):
    dev = torch.device("cuda:0")
    n = max(t0 + c for t0, c in ranges)
    x = _bits((n, h_loc, D), 200 + world).to(dev)
    dst = [_poisoned((max(c, 1), h_dst, D), dev) for _, c in ranges]
    binding.regenvc_ulysses_gather_heads(x, dst, [t for t, _ in ranges], [c for _, c in ranges], h_dst, head0)
    torch.cuda.synchronize()
    for r, (t0, c) in enumerate(ranges):
        got = dst[r].view(torch.int16)
        want = torch.full_like(got, POISON)
        want[:c, head0:head0 + h_loc] = x[t0:t0 + c].view(torch.int16)
        assert torch.equal(got, want), f"destination {r}"


def test_scatter_then_gather_is_the_identity_for_a_whole_group():
    dev = torch.device("cuda:0")
    U, h, shards = 4, 8, [31, 30, 30, 30]
    xs = [_bits((n, h, D), 300 + i).to(dev) for i, n in enumerate(shards)]
    t0 = np.concatenate([[0], np.cumsum(shards)]).tolist()
    blocks = [_poisoned((t0[-1], h // U, D), dev) for _ in range(U)]
    for i, x in enumerate(xs):
        binding.regenvc_ulysses_scatter_heads(x, blocks, t0[i])
    back = [_poisoned((n, h, D), dev) for n in shards]
    for u in range(U):
        binding.regenvc_ulysses_gather_heads(blocks[u], back, t0[:-1], shards, h, u * (h // U))
    torch.cuda.synchronize()
    for x, y in zip(xs, back):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))


def test_resharding_argument_checks():
    L = binding.lib()
    import ctypes
    a = 0x100000
    one = (ctypes.c_void_p * 1)(a + 0x100000)
    two = (ctypes.c_void_p * 2)(a + 0x100000, None)
    i1 = (ctypes.c_int * 2)(0, 0)
    f, g = L.regenvc_ulysses_scatter_heads, L.regenvc_ulysses_gather_heads
    assert f(None, one, 1, 4, 0, 2, 128, None) == binding.ERR_NULL_POINTER
    assert f(a, two, 2, 4, 0, 2, 128, None) == binding.ERR_NULL_POINTER
    assert f(a, one, 0, 4, 0, 2, 128, None) == binding.ERR_BAD_SHAPE
    assert f(a, one, 17, 4, 0, 34, 128, None) == binding.ERR_BAD_SHAPE
    assert f(a, two, 2, 4, 0, 3, 128, None) == binding.ERR_BAD_SHAPE      # heads not divisible
    assert f(a, one, 1, 4, 0, 2, 64, None) == binding.ERR_UNSUPPORTED
    assert f(a + 2, one, 1, 4, 0, 2, 128, None) == binding.ERR_MISALIGNED
    same = (ctypes.c_void_p * 1)(a)
    assert f(a, same, 1, 4, 0, 2, 128, None) == binding.ERR_ALIASING
    assert g(a, one, None, i1, 1, 2, 2, 0, 128, None) == binding.ERR_NULL_POINTER
    assert g(a, one, i1, i1, 1, 2, 1, 0, 128, None) == binding.ERR_BAD_SHAPE   # destination narrower than source
    assert g(a, one, i1, i1, 1, 2, 4, 3, 128, None) == binding.ERR_BAD_SHAPE   # head range past the destination


@pytest.mark.parametrize("grid,h,U,R", [
    ((2, 9, 14), 4, 2, 1), ((2, 9, 14), 2, 1, 2), ((3, 10, 13), 4, 2, 2), ((2, 16, 20), 8, 4, 2),
    ((1, 7, 11), 6, 3, 3),
])
def test_usp_on_one_gpu_equals_unsharded_attention(grid, h, U, R):
    T, H, W = grid
    N = T * H * W
    rng = np.random.default_rng(8000 + N + 10 * U + R)
    q = synth.from_f32(rng.standard_normal((N, h, D)))
    k = synth.from_f32(rng.standard_normal((N, h, D)) * 1.5)
    v = synth.from_f32(rng.standard_normal((N, h, D)))
    dev = torch.device("cuda:0")
    layout = usp.UspLayout(U * R, U, R, N, h)
    outs = usp.usp_attention_one_gpu(q.to(dev), k.to(dev), v.to(dev), T, H, W, layout)
    assert binding.regenvc_device_status() == 0
    assert [o.shape[0] for o in outs] == [layout.shard(g)[1] for g in range(layout.world)]
    got = torch.cat(outs).cpu()
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W)
    assert_parity(f64(got), ref, float(v.float().abs().max()), f"usp {grid} U={U} R={R}")
    full = torch.empty((N, h, D), dtype=torch.bfloat16, device=dev)
    binding.regenvc_attn_forward(q.to(dev), k.to(dev), v.to(dev), full, T, H, W)
    if R == 1:
        assert torch.equal(got, full.cpu())  # heads are independent: resharding alone changes no bit
    else:
        assert float((got.float() - full.cpu().float()).abs().max()) <= 2 ** -7 * float(v.float().abs().max())


def test_usp_paper_degrees_on_a_window_slice():
    """U = 4, R = 2 (the paper's 8-GPU setting) on a 2-frame slice of the 480x832 grid with 12 heads."""
    T, H, W, h = 2, 30, 52, 12
    N = T * H * W
    w = synth.Workload(name="slice", seed=77, T=T, H=H, W=W, n_heads=h, layers=1)
    q, k, v = synth.self_inputs(w)
    dev = torch.device("cuda:0")
    layout = usp.UspLayout(8, 4, 2, N, h)
    got = torch.cat(usp.usp_attention_one_gpu(q.to(dev), k.to(dev), v.to(dev), T, H, W, layout)).cpu()
    assert binding.regenvc_device_status() == 0
    rows = synth.sample_rows(N, H, W, seed=77, n_random=64)
    for a in (0, 5, 11):
        ref = oracle.self_attn_head(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W, a, rows=rows)
        assert_parity(got[rows, a].double().numpy(), ref, float(v.float().abs().max()), f"usp 4x2 head {a}")


class _ThreadFabric:
    """In-process stand-in for the process-group calls UspAttention makes, for ranks that run as host THREADS on
    one GPU: messages are device tensors handed over through FIFO queues per (source, destination).  All waiting
    happens on the host, never inside a kernel, and every rank's kernels go to the same stream."""

    def __init__(self, world):
        import queue
        self.q = {(s, d): queue.Queue() for s in range(world) for d in range(world)}

    def endpoint(self, rank):
        return _ThreadDist(self, rank)


class _ThreadDist:
    isend, irecv = "isend", "irecv"

    class _Req:
        def __init__(self, fn):
            self.fn = fn

        def wait(self):
            self.fn()

    def __init__(self, fabric, rank):
        self.f, self.rank = fabric, rank

    def all_to_all_single(self, recv, send, output_split_sizes, input_split_sizes, group):
        at = 0
        for peer, n in zip(group, input_split_sizes):
            self.f.q[(self.rank, peer)].put(send[at:at + n].clone())
            at += n
        assert at == send.shape[0]
        at = 0
        for peer, n in zip(group, output_split_sizes):
            msg = self.f.q[(peer, self.rank)].get(timeout=120)
            assert msg.shape[0] == n
            recv[at:at + n].copy_(msg)
            at += n
        assert at == recv.shape[0]

    def P2POp(self, op, tensor, peer, group):
        return (op, tensor, peer)

    def batch_isend_irecv(self, ops):
        reqs = []
        for op, tensor, peer in ops:
            if op == self.isend:
                self.f.q[(self.rank, peer)].put(tensor.clone())
                reqs.append(self._Req(lambda: None))
            else:
                reqs.append(self._Req(lambda t=tensor, p=peer: t.copy_(self.f.q[(p, self.rank)].get(timeout=120))))
        return reqs


@pytest.mark.parametrize("grid,h,U,R", [((2, 9, 14), 4, 1, 1), ((2, 9, 14), 4, 2, 1), ((3, 10, 13), 2, 1, 2),
                                        ((2, 16, 20), 8, 2, 2), ((2, 12, 26), 12, 4, 2)])
def test_per_rank_driver_with_the_cuda_kernels_on_host_threads(grid, h, U, R):
    """usp.UspAttention with usp.CudaOps -- the per-rank driver exactly as a multi-GPU job runs it: packing by the
    resharding kernels, exchange, block-wise attention, merge, exchange back -- for every rank of a U x R layout,
    each rank a host thread on this one GPU.  Only the transport under all_to_all_single / batch_isend_irecv is
    replaced (queues of device tensors instead of NCCL); the joined output shards must equal unsharded attention."""
    import threading

    T, H, W = grid
    N, world = T * H * W, U * R
    rng = np.random.default_rng(8100 + N + 10 * U + R)
    q = synth.from_f32(rng.standard_normal((N, h, D)))
    k = synth.from_f32(rng.standard_normal((N, h, D)) * 1.5)
    v = synth.from_f32(rng.standard_normal((N, h, D)))
    dev = torch.device("cuda:0")
    layout = usp.UspLayout(world, U, R, N, h)
    fabric = _ThreadFabric(world)
    outs, errs = [None] * world, []

    def run(rank):
        try:
            torch.cuda.set_device(dev)
            t0, cnt = layout.shard(rank)
            ql, kl, vl = (x[t0:t0 + cnt].contiguous().to(dev) for x in (q, k, v))
            attn = usp.UspAttention(layout, rank, layout.ulysses_group(rank), layout.ring_group(rank),
                                    ops=usp.CudaOps(), dist=fabric.endpoint(rank))
            outs[rank] = attn(ql, kl, vl, T, H, W).cpu()
        except Exception as ex:  # surfaced below: a dead thread would leave its peers waiting on their queues
            errs.append((rank, repr(ex)))

    threads = [threading.Thread(target=run, args=(g,)) for g in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errs, errs
    assert all(o is not None for o in outs)
    assert binding.regenvc_device_status() == 0
    got = torch.cat(outs)
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W)
    assert_parity(f64(got), ref, float(v.float().abs().max()), f"per-rank driver U={U} R={R}")
    emu = torch.cat(usp.usp_attention_one_gpu(q.to(dev), k.to(dev), v.to(dev), T, H, W, layout)).cpu()
    assert torch.equal(got, emu)  # same kernels on the same data in the same order as the one-thread emulation


def test_resharding_bandwidth_report(capsys):
    """HBM-bound copies: prints the achieved rate at the 480x832 window shape (run with -s to see it) and checks
    that it is at least a sizeable fraction of the memory system's (a regression guard, not a tuning target)."""
    dev = torch.device("cuda:0")
    U, n_loc, h = 4, 1365, 12   # one rank's shard of the 10 920-token window, Ulysses degree 4
    xs = [_bits((n_loc, h, D), 900 + i).to(dev) for i in range(8)]  # 8 x 4.2 MB sources, rotated
    blocks = [_poisoned((U * n_loc, h // U, D), dev) for _ in range(U)]
    big = _bits((31200, 10, D), 950).to(dev)    # a head shard of the 77-frame clip (80 MB)
    outs = [_poisoned((3900, 40, D), dev) for _ in range(4)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        e0.record()
        for i in range(reps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e-3

    t_s = timed(lambda i: binding.regenvc_ulysses_scatter_heads(xs[i % 8], blocks, 0), 200)
    t_g = timed(lambda i: binding.regenvc_ulysses_gather_heads(big, outs, [0, 3900, 7800, 11700], [3900] * 4, 40,
                                                               10 * (i % 4)), 50)
    gbs_s = 2 * xs[0].numel() * 2 / t_s / 1e9
    gbs_g = 2 * 4 * 3900 * 10 * D * 2 / t_g / 1e9
    with capsys.disabled():
        print(f"\nscatter_heads 4.2 MB shard: {t_s * 1e6:.1f} us, {gbs_s:.0f} GB/s (read + write)")
        print(f"gather_heads 40 MB of an 80 MB head shard: {t_g * 1e6:.1f} us, {gbs_g:.0f} GB/s (read + write)")
    assert gbs_g > 1500.0
