"""Unified sequence parallelism around the attention kernels (Sec. 3.5: Ulysses x Ring).

The token sequence is cut into ``world = ulysses * ring`` contiguous shards, one per GPU.  Inside a Ulysses group
(``ulysses`` GPUs that hold consecutive shards) an all-to-all turns the sequence sharding into a head sharding, so
each GPU holds one *ring block* of tokens (the group's shards joined) for ``n_heads / ulysses`` heads.  The ring
blocks of keys and values then travel around the ``ring`` GPUs that hold the same heads; every GPU computes the
attention of its query block against each key/value block (``regenvc_attn_partial``) and merges the partial
results exactly (``regenvc_attn_merge``).  A second all-to-all restores the sequence sharding of the output.

This module holds
  * :class:`UspLayout` -- who holds which tokens and heads, and the ring schedule (pure host arithmetic);
  * :func:`usp_attention_one_gpu` -- every rank's work executed one rank after another on the current GPU,
    with the destination buffers of the resharding kernels standing in for the peers' memory;
  * :class:`UspAttention` -- the per-rank driver over ``torch.distributed`` (NCCL all-to-all for the two
    resharding steps with the library's kernels doing the packing, point-to-point transfers for the ring).

Only the data movement and the order of calls live here; all arithmetic is in the CUDA kernels.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple


@dataclass(frozen=True)
class UspLayout:
    """Token and head ownership for ``world = ulysses * ring`` ranks.

    Rank ``g`` has Ulysses index ``u = g % ulysses`` and ring index ``r = g // ulysses``; shards are contiguous
    token ranges in rank order (sizes differ by at most one token)."""
    world: int
    ulysses: int
    ring: int
    n_tokens: int
    n_heads: int

    def __post_init__(self):
        if self.ulysses < 1 or self.ring < 1 or self.world != self.ulysses * self.ring:
            raise ValueError("world must equal ulysses * ring")
        if self.n_heads < 1 or self.n_heads % self.ulysses != 0:
            raise ValueError("the head count must be a multiple of the Ulysses degree")
        if self.n_tokens < self.world:
            raise ValueError("need at least one token per rank")
        if self.ulysses > 16 or self.ring > 8:
            raise ValueError("at most 16 Ulysses peers and 8 ring blocks")

    # ---- coordinates
    def coords(self, rank: int) -> Tuple[int, int]:
        self._check_rank(rank)
        return rank % self.ulysses, rank // self.ulysses

    def rank_of(self, u: int, r: int) -> int:
        if not (0 <= u < self.ulysses and 0 <= r < self.ring):
            raise ValueError("coordinates out of range")
        return r * self.ulysses + u

    def ulysses_group(self, rank: int) -> List[int]:
        _, r = self.coords(rank)
        return [self.rank_of(u, r) for u in range(self.ulysses)]

    def ring_group(self, rank: int) -> List[int]:
        u, _ = self.coords(rank)
        return [self.rank_of(u, r) for r in range(self.ring)]

    # ---- ownership
    def shard(self, rank: int) -> Tuple[int, int]:
        """(first token, token count) of the sequence shard of ``rank``."""
        self._check_rank(rank)
        base, rem = divmod(self.n_tokens, self.world)
        return rank * base + min(rank, rem), base + (1 if rank < rem else 0)

    def block(self, r: int) -> Tuple[int, int]:
        """(first token, token count) of ring block ``r``: the shards of its Ulysses group joined."""
        first, _ = self.shard(self.rank_of(0, r))
        last0, last_n = self.shard(self.rank_of(self.ulysses - 1, r))
        return first, last0 + last_n - first

    def heads(self, u: int) -> Tuple[int, int]:
        """(first head, head count) held by Ulysses index ``u`` after the first all-to-all."""
        per = self.n_heads // self.ulysses
        if not 0 <= u < self.ulysses:
            raise ValueError("Ulysses index out of range")
        return u * per, per

    # ---- ring schedule
    def ring_source(self, r: int, step: int) -> int:
        """Ring block whose keys/values ring member ``r`` holds at ``step`` (0 = its own)."""
        return (r - step) % self.ring

    def ring_next(self, r: int) -> int:
        return (r + 1) % self.ring

    def ring_prev(self, r: int) -> int:
        return (r - 1) % self.ring

    def _check_rank(self, rank: int):
        if not 0 <= rank < self.world:
            raise ValueError("rank out of range")


class CudaOps:
    """The kernels the drivers below call, through the C ABI (there is no other implementation)."""

    def __init__(self):
        import torch
        from . import binding
        binding.lib()  # fails loudly when the CUDA library has not been built
        self.torch, self.b = torch, binding

    def empty(self, shape, dtype, like):
        return self.torch.empty(shape, dtype=dtype, device=like.device)

    def scatter_heads(self, x_local, dst, dst_token0):
        self.b.regenvc_ulysses_scatter_heads(x_local, dst, dst_token0)

    def gather_heads(self, x_heads, dst, token0, n_tokens, n_heads_dst, dst_head0):
        self.b.regenvc_ulysses_gather_heads(x_heads, dst, token0, n_tokens, n_heads_dst, dst_head0)

    def forward(self, q, k, v, out, T, H, W, theta):
        self.b.regenvc_attn_forward(q, k, v, out, T, H, W, theta)

    def partial(self, q, k, v, T, H, W, q_token0, kv_token0, theta):
        n_q, h, d = q.shape
        o = self.torch.empty((n_q, h, d), dtype=self.torch.float32, device=q.device)
        ml = self.torch.empty((n_q, h, 2), dtype=self.torch.float32, device=q.device)
        self.b.regenvc_attn_partial(q, k, v, o, ml, T, H, W, q_token0, kv_token0, theta)
        return o, ml

    def merge(self, parts, out):
        self.b.regenvc_attn_merge([p[0] for p in parts], [p[1] for p in parts], out)


def _block_attention(ops, layout: UspLayout, r: int, q_blk, kv_of_step, T, H, W, theta):
    """Attention of ring member ``r``'s query block against every key/value block, in ring order.
    ``kv_of_step(step)`` returns the (k, v) block the member holds at that step."""
    q0, _ = layout.block(r)
    out = ops.empty(tuple(q_blk.shape), q_blk.dtype, q_blk)
    if layout.ring == 1:
        k, v = kv_of_step(0)
        ops.forward(q_blk, k, v, out, T, H, W, theta)
        return out
    parts = []
    for step in range(layout.ring):
        k, v = kv_of_step(step)
        kv0, _ = layout.block(layout.ring_source(r, step))
        parts.append(ops.partial(q_blk, k, v, T, H, W, q0, kv0, theta))
    ops.merge(parts, out)
    return out


def usp_attention_one_gpu(q, k, v, T: int, H: int, W: int, layout: UspLayout, rope_theta: float = 10000.0,
                          ops=None) -> list:
    """Runs the work of all ``layout.world`` ranks on the current GPU, one rank after another.

    ``q, k, v``: the whole [T*H*W, heads, head_dim] tensors; each rank's shard is cut out first, and from then on
    a rank only touches its own shard and the buffers the scheme gives it.  Returns the per-rank output shards
    (their concatenation is the attention output)."""
    ops = ops or CudaOps()
    n, h, d = q.shape
    if n != T * H * W or n != layout.n_tokens or h != layout.n_heads:
        raise ValueError("tensor shape does not match the layout")
    U, R = layout.ulysses, layout.ring
    h_loc = h // U
    local = [[x[t0:t0 + cnt].contiguous() for x in (q, k, v)] for t0, cnt in map(layout.shard, range(layout.world))]

    # first all-to-all: every member of a Ulysses group writes its tokens into the block buffers of all members
    blocks = [[None] * U for _ in range(R)]
    for r in range(R):
        b0, bn = layout.block(r)
        bufs = [[ops.empty((bn, h_loc, d), q.dtype, q) for _ in range(3)] for _ in range(U)]
        for u_src in range(U):
            rank = layout.rank_of(u_src, r)
            t0, _ = layout.shard(rank)
            for i in range(3):
                ops.scatter_heads(local[rank][i], [bufs[u][i] for u in range(U)], t0 - b0)
        for u in range(U):
            blocks[r][u] = bufs[u]

    # ring + merge, then the second all-to-all back to sequence shards
    outs = [ops.empty((layout.shard(g)[1], h, d), q.dtype, q) for g in range(layout.world)]
    for r in range(R):
        b0, _ = layout.block(r)
        for u in range(U):
            q_blk = blocks[r][u][0]

            def kv_of_step(step, u=u, r=r):
                src = layout.ring_source(r, step)
                return blocks[src][u][1], blocks[src][u][2]

            o_blk = _block_attention(ops, layout, r, q_blk, kv_of_step, T, H, W, rope_theta)
            group = layout.ulysses_group(layout.rank_of(u, r))
            ranges = [layout.shard(g) for g in group]
            ops.gather_heads(o_blk, [outs[g] for g in group], [t0 - b0 for t0, _ in ranges],
                             [cnt for _, cnt in ranges], h, layout.heads(u)[0])
    return outs


def make_groups(layout: UspLayout, rank: int, dist=None):
    """Creates every Ulysses group and every ring group (all ranks must call this, in the same order) and returns
    this rank's (ulysses_group, ring_group) process groups."""
    if dist is None:
        import torch.distributed as dist
    mine_u = mine_r = None
    for r in range(layout.ring):
        ranks = [layout.rank_of(u, r) for u in range(layout.ulysses)]
        g = dist.new_group(ranks)
        if rank in ranks:
            mine_u = g
    for u in range(layout.ulysses):
        ranks = [layout.rank_of(u, r) for r in range(layout.ring)]
        g = dist.new_group(ranks)
        if rank in ranks:
            mine_r = g
    return mine_u, mine_r


class UspAttention:
    """Per-rank driver: ``out_local = UspAttention(...)(q_local, k_local, v_local, T, H, W)``.

    The two resharding steps are ``all_to_all_single`` calls whose send/receive buffers are packed and unpacked by
    the library's resharding kernels; the ring moves whole key/value blocks with point-to-point transfers that
    are posted before the partial attention of the block at hand, so that transfer and compute overlap."""

    def __init__(self, layout: UspLayout, rank: int, ulysses_pg, ring_pg, ops=None, dist=None):
        if dist is None:
            import torch.distributed as dist
        self.layout, self.rank, self.dist = layout, rank, dist
        self.u, self.r = layout.coords(rank)
        self.ulysses_pg, self.ring_pg = ulysses_pg, ring_pg
        self.ops = ops or CudaOps()

    def _to_heads(self, x_local):
        """[n_local, h, d] of this rank -> [block tokens, h / U, d] (first all-to-all)."""
        L, U = self.layout, self.layout.ulysses
        n_loc, h, d = x_local.shape
        h_loc = h // U
        if U == 1:
            return x_local
        send = self.ops.empty((U * n_loc, h_loc, d), x_local.dtype, x_local)
        self.ops.scatter_heads(x_local, [send[u * n_loc:(u + 1) * n_loc] for u in range(U)], 0)
        rows = [L.shard(g)[1] for g in L.ulysses_group(self.rank)]
        recv = self.ops.empty((sum(rows), h_loc, d), x_local.dtype, x_local)
        self.dist.all_to_all_single(recv, send, output_split_sizes=rows, input_split_sizes=[n_loc] * U,
                                    group=self.ulysses_pg)
        return recv

    def _to_tokens(self, o_blk, n_heads):
        """[block tokens, h / U, d] -> [n_local, h, d] of this rank (second all-to-all)."""
        L, U = self.layout, self.layout.ulysses
        if U == 1:
            return o_blk
        _, h_loc, d = o_blk.shape
        n_loc = L.shard(self.rank)[1]
        rows = [L.shard(g)[1] for g in L.ulysses_group(self.rank)]
        recv = self.ops.empty((U * n_loc, h_loc, d), o_blk.dtype, o_blk)
        self.dist.all_to_all_single(recv, o_blk, output_split_sizes=[n_loc] * U, input_split_sizes=rows,
                                    group=self.ulysses_pg)
        out = self.ops.empty((n_loc, n_heads, d), o_blk.dtype, o_blk)
        for u in range(U):
            self.ops.gather_heads(recv[u * n_loc:(u + 1) * n_loc], [out], [0], [n_loc], n_heads, L.heads(u)[0])
        return out

    def __call__(self, q_local, k_local, v_local, T: int, H: int, W: int, rope_theta: float = 10000.0):
        L, dist = self.layout, self.dist
        n_loc, h, d = q_local.shape
        if n_loc != L.shard(self.rank)[1] or h != L.n_heads or T * H * W != L.n_tokens:
            raise ValueError("tensor shape does not match the layout")
        q_blk, k_blk, v_blk = (self._to_heads(x) for x in (q_local, k_local, v_local))
        ring_ranks = L.ring_group(self.rank)
        nxt, prv = ring_ranks[L.ring_next(self.r)], ring_ranks[L.ring_prev(self.r)]
        held = {"kv": (k_blk, v_blk), "pending": None, "incoming": None}

        def kv_of_step(step):
            if held["pending"] is not None:  # the block posted during the previous step has to be here now
                for req in held["pending"]:
                    req.wait()
                held["kv"], held["pending"] = held["incoming"], None
            k_cur, v_cur = held["kv"]
            if step + 1 < L.ring:
                rows = L.block(L.ring_source(self.r, step + 1))[1]
                k_in = self.ops.empty((rows,) + tuple(k_cur.shape[1:]), k_cur.dtype, k_cur)
                v_in = self.ops.empty((rows,) + tuple(v_cur.shape[1:]), v_cur.dtype, v_cur)
                ops_list = [dist.P2POp(dist.isend, k_cur, nxt, self.ring_pg),
                            dist.P2POp(dist.isend, v_cur, nxt, self.ring_pg),
                            dist.P2POp(dist.irecv, k_in, prv, self.ring_pg),
                            dist.P2POp(dist.irecv, v_in, prv, self.ring_pg)]
                held["pending"], held["incoming"] = dist.batch_isend_irecv(ops_list), (k_in, v_in)
            return k_cur, v_cur

        o_blk = _block_attention(self.ops, L, self.r, q_blk, kv_of_step, T, H, W, rope_theta)
        return self._to_tokens(o_blk, h)
