#!/usr/bin/env python
"""Benchmark of the fused 3D-RoPE attention path on seeded synthetic tensors.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
                    [--sustain-seconds S] [--usp UxR]

One "step" is one pass of the whole hot path over one window: the
self-attention call (key/value preparation pass + attention kernel) followed by
one cross-attention call per conditioning sequence of the workload, on
conditioning operands that were prepared once before the timed region (the
paper computes the conditioning keys/values once per sequence, Sec. 3.9; the
step with that preparation inside every call is timed as well).  At N = 1
the workload is the 480x832 window (7x30x52 = 10920 tokens, 12 heads x 128,
plus 512 conditioning tokens), the shape the tensor-peak target is quoted on.
With N > 1 (one process per GPU under torchrun; without a launcher the script
starts the N ranks itself) every rank runs its own window (heads and windows
are independent: no data-path collective, weak scaling).  After the K timed
steps the same step loop is repeated for at least S seconds (default 4) with
the clocks sampled throughout, which gives the power-capped, sustained
figures next to the burst ones.  --usp UxR instead spreads ONE window over
U*R ranks as Ulysses x Ring (strong scaling, the paper's decomposition).

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2607_28144_b200 import synth

NOMINAL_BF16_TFLOPS = 2250.0  # dense bf16/fp16 datasheet figure, context only
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
PAPER_CONTEXT = ("paper: 972 ms per 25-frame window (24 fps) for the WHOLE decoder on 8 consumer-class GPUs; "
                 "it reports no attention-only number")
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the self-attention kernel at the 480x832 window
# shape, from one ncu capture of that launch (101.6 MB read + 19.7 MB written; the rest of the 33.5 MB output is
# still in L2 when the kernel ends).
ATTN_KERNEL_DRAM_TRAFFIC_BYTES = {"window_480x832": 121.3e6}
N_BUFFER_SETS = 4
KERNEL_BITS = 0  # --kernel: debug bits that force (8) or forbid (16) the attention kernel on pairs of thread blocks


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as ex:  # NVML missing: report that instead of clocks
            self.nv = None
            self.err = repr(ex)

    _BITS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
             0x80: "hw_power_brake_slowdown"}

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                r = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self._BITS.items():
                    if r & bit:
                        self.reasons.add(name)
                self.power.append(self.nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            time.sleep(0.001)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if self.nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "error": self.err}
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None,
                "power_w_median": statistics.median(self.power) if self.power else None}


def rank_seed_offset(set_index: int, rank: int) -> int:
    """Seed offset of input set `set_index` on `rank`: every rank runs its own window (distinct inputs)."""
    return 100 * set_index + 7 * rank


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_tflops(world: int, flops_per_step: float, ms_per_step: float) -> float:
    """Weak scaling: every rank processes one window per step; the job's rate is all windows over the slowest rank's time."""
    return world * flops_per_step / (ms_per_step * 1e-3) / 1e12


def self_attention_kernel_name(w: synth.Workload, sm_count: int) -> str:
    """Which kernel the library enqueues for this workload's self-attention call (its rule, restated): long key
    sequences with at least one full round of work items run on pairs of thread blocks."""
    n_tiles = -(-w.n_tokens // 128)
    n_items = -(-w.n_tokens // 256) * w.n_heads
    pair = KERNEL_BITS == 8 or (KERNEL_BITS == 0 and n_tiles >= 32 and n_items >= sm_count // 2)
    return ("attn_pair_kernel" if pair else "attn_pipelined_kernel") + " (self-attention)"


def step_flops(w: synth.Workload) -> float:
    return w.self_flops() + sum(w.cross_flops(n) for n in w.cross_kv)


# ------------------------------------------------------------------------------------------------ oracle legs
def oracle_sample(w: synth.Workload, heads, q, k, v, cross, rows=None):
    """Times the fp64 oracle, as it stands, on `heads` x `rows` (None = all query rows) of one step.
    Returns (seconds, flops)."""
    import oracle

    qb, kb, vb = synth.bits(q), synth.bits(k), synth.bits(v)
    cb = [(synth.bits(a), synth.bits(b)) for a, b in cross]
    t0 = time.perf_counter()
    for a in heads:
        oracle.self_attn_head(qb, kb, vb, w.T, w.H, w.W, a, w.theta, rows=rows)
        for (ck, cv) in cb:
            oracle.cross_attn_head(qb, ck, cv, a, rows=rows)
    dt = time.perf_counter() - t0
    n_rows = w.n_tokens if rows is None else len(rows)
    fl = len(heads) * (step_flops(w) / w.n_heads) * (n_rows / w.n_tokens)
    return dt, fl


def run_reference(args, w: synth.Workload):
    """--impl reference: the oracle on the host cores.  Each step is a bounded sample of one step of the
    workload (head 0, evenly spaced query rows, self + cross), sized so that the whole run takes about two
    minutes whatever --steps / --warmup are."""
    import oracle

    oracle.build()
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    q, k, v = synth.self_inputs(w)
    cross = [synth.cross_inputs(w, n) for n in w.cross_kv]
    heads = [0]
    probe_rows = np.linspace(0, w.n_tokens - 1, num=min(256, w.n_tokens)).astype(np.int64)
    dt, fl = oracle_sample(w, heads, q, k, v, cross, probe_rows)
    dt, fl = oracle_sample(w, heads, q, k, v, cross, probe_rows)
    rows_per_s = len(probe_rows) / dt
    budget_s = 120.0 / (args.steps + args.warmup)
    n_rows = int(min(w.n_tokens, max(32, budget_s * rows_per_s)))
    rows = np.linspace(0, w.n_tokens - 1, num=n_rows).astype(np.int64)
    for _ in range(args.warmup):
        oracle_sample(w, heads, q, k, v, cross, rows)
    t_total, f_total = 0.0, 0.0
    for _ in range(args.steps):
        dt, fl = oracle_sample(w, heads, q, k, v, cross, rows)
        t_total += dt
        f_total += fl
    tflops = f_total / t_total / 1e12
    ms_full_step = step_flops(w) / (tflops * 1e12) * 1e3
    line = {
        "impl": "reference", "metric": "attention bf16 TFLOP/s", "value": tflops, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_full_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "grid_THW": [w.T, w.H, w.W], "tokens": w.n_tokens, "heads": w.n_heads,
                   "head_dim": w.head_dim, "cross_kv": list(w.cross_kv), "layers": w.layers, "denoise_steps": w.steps,
                   "note": "ms_per_step is the sampled rate extrapolated to the full step"},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
                         "sample": f"per step: head 0 of {w.n_heads}, {n_rows} evenly spaced query rows of "
                                   f"{w.n_tokens}, self + cross"},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "ms_per_window": ms_full_step * w.layers * w.steps,
        "context": PAPER_CONTEXT,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------ CUDA path
def _events(n):
    return [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]


def _setup_ranks(args):
    """Rank bookkeeping.  Fails loudly when fewer ranks or GPUs than --gpus come up."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torchrun --nproc-per-node {args.gpus}")
    if torch.cuda.device_count() <= local:
        raise SystemExit(f"rank {rank} needs cuda:{local} but only {torch.cuda.device_count()} GPU(s) are visible")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist, seen = None, 1
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
        ones = torch.ones((), dtype=torch.int32, device=dev)
        dist.all_reduce(ones)
        seen = int(ones.item())
        if seen != args.gpus or dist.get_world_size() != args.gpus:
            raise SystemExit(f"--gpus {args.gpus} but the communicator has {seen} rank(s)")
    return rank, world, local, dev, dist, seen


def time_producer_fusion(binding, w: synth.Workload, dev, stream, n=20):
    """Times, with CUDA events on `stream`, (a) the fused producer + attention on its operands and (b) the same
    block computed as projection-then-attention with library kernels in front of the ordinary call."""
    C, N, h = w.n_heads * w.head_dim, w.n_tokens, w.n_heads
    x, wq, b, gq, gk, eps = (t.to(dev) if torch.is_tensor(t) else t for t in synth.block_inputs(w))
    q_rot, prepared = binding.regenvc_qkv_rope_project(x, wq, b, gq, gk, eps, w.T, w.H, w.W, h, w.theta, stream=stream)
    out = torch.empty((N, h, w.head_dim), dtype=torch.bfloat16, device=dev)
    b16 = b.to(torch.bfloat16)

    def producer():
        binding.regenvc_qkv_rope_project(x, wq, b, gq, gk, eps, w.T, w.H, w.W, h, w.theta, q_rot=q_rot,
                                         prepared=prepared, stream=stream)

    def attn_prepared():
        binding.regenvc_attn_forward_prepared(q_rot, prepared, N, out, stream)

    def library_projection():
        y = torch.addmm(b16, x, wq.t()).float()
        q, k = y[:, :C], y[:, C:2 * C]
        q = (q * torch.rsqrt(q.pow(2).mean(-1, keepdim=True) + eps) * gq).to(torch.bfloat16).view(N, h, w.head_dim)
        k = (k * torch.rsqrt(k.pow(2).mean(-1, keepdim=True) + eps) * gk).to(torch.bfloat16).view(N, h, w.head_dim)
        return q, k, y[:, 2 * C:].to(torch.bfloat16).view(N, h, w.head_dim)

    q, k, v = (t.contiguous() for t in library_projection())

    def attn_plain():
        binding.regenvc_attn_forward(q, k, v, out, w.T, w.H, w.W, w.theta, stream)

    def timed(fn):
        for _ in range(3):
            fn()
        evs = _events(n)
        for a, bb in evs:
            a.record(stream)
            fn()
            bb.record(stream)
        torch.cuda.synchronize()
        return statistics.mean(a.elapsed_time(bb) for a, bb in evs)

    wo, bo = (t.to(dev) for t in synth.out_proj_inputs(w))
    y = torch.empty((N, C), dtype=torch.bfloat16, device=dev)
    bo16 = bo.to(torch.bfloat16)
    out2d = out.view(N, C)

    def out_proj():
        binding.regenvc_out_project(out, wo, bo, y=y, stream=stream)

    t_prod, t_attn_p = timed(producer), timed(attn_prepared)
    t_oproj, t_oproj_lib = timed(out_proj), timed(lambda: torch.addmm(bo16, out2d, wo.t()))
    t_gemm = timed(lambda: torch.addmm(b16, x, wq.t()))
    t_lib, t_attn = timed(library_projection), timed(attn_plain)
    flops = 2.0 * N * 3 * C * C
    return {"producer_ms": t_prod, "producer_tflops": flops / (t_prod * 1e-3) / 1e12,
            "attention_on_prepared_operands_ms": t_attn_p, "fused_ms": t_prod + t_attn_p,
            "library_gemm_only_ms": t_gemm, "library_projection_norm_ms": t_lib,
            "attention_with_preparation_pass_ms": t_attn, "unfused_ms": t_lib + t_attn,
            "out_project_ms": t_oproj, "out_project_tflops": 2.0 * N * C * C / (t_oproj * 1e-3) / 1e12,
            "library_out_project_gemm_ms": t_oproj_lib, "block_attention_part_ms": t_prod + t_attn_p + t_oproj,
            "note": "fused = regenvc_qkv_rope_project + regenvc_attn_forward_prepared (no preparation pass, no "
                    "bf16 round trip of q, k, v); unfused = library GEMM + eager norm kernels + regenvc_attn_forward; "
                    "block_attention_part = fused + regenvc_out_project (y = o W_o^T + b_o, bf16)"}


def run_ours(args, w: synth.Workload):
    global KERNEL_BITS
    KERNEL_BITS = {"auto": 0, "pair": 8, "single": 16}[args.kernel]
    from paper_2607_28144_b200 import binding, build

    build.build()
    rank, world, local, dev, dist, ranks_seen = _setup_ranks(args)
    if KERNEL_BITS:
        binding.regenvc_debug_set_phases(3 | KERNEL_BITS)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # inputs: N_BUFFER_SETS distinct sets so that consecutive steps do not find their inputs in L2
    sets = []
    for i in range(N_BUFFER_SETS):
        wi = synth.Workload(**{**w.__dict__, "seed": w.seed + rank_seed_offset(i, rank)})
        q, k, v = synth.self_inputs(wi)
        cross = [synth.cross_inputs(wi, n) for n in w.cross_kv]
        sets.append({"q": q.to(dev), "k": k.to(dev), "v": v.to(dev),
                     "cross": [(a.to(dev), b.to(dev)) for a, b in cross],
                     "out": torch.empty_like(q, device=dev), "outc": [torch.empty_like(q, device=dev) for _ in cross],
                     # the conditioning keys/values are computed once per sequence (Sec. 3.9): their operand form is
                     # prepared here, once, and every timed step runs the cross-attention call on it
                     "prepared": [binding.regenvc_cross_kv_prepare(a.to(dev), b.to(dev)) for a, b in cross],
                     # a workspace of its own, used only where the attention kernel is timed alone: the operands
                     # prepared from this set's k and v stay in it between launches
                     "ws": torch.empty((binding.regenvc_workspace_bytes(w.n_tokens, w.n_heads),), dtype=torch.uint8,
                                       device=dev)})
    host0 = None
    stream = torch.cuda.Stream(device=dev)

    def step(s):
        binding.regenvc_attn_forward(s["q"], s["k"], s["v"], s["out"], w.T, w.H, w.W, w.theta, stream)
        for prep, n_kv, oc in zip(s["prepared"], w.cross_kv, s["outc"]):
            binding.regenvc_cross_attn_forward_prepared(s["q"], prep, n_kv, oc, stream)

    def step_one_call_cross(s):
        binding.regenvc_attn_forward(s["q"], s["k"], s["v"], s["out"], w.T, w.H, w.W, w.theta, stream)
        for (ck, cv), oc in zip(s["cross"], s["outc"]):
            binding.regenvc_cross_attn_forward(s["q"], ck, cv, oc, stream)

    def self_call(s):
        binding.regenvc_attn_forward(s["q"], s["k"], s["v"], s["out"], w.T, w.H, w.W, w.theta, stream)

    def kernel_only_loop(n, per_launch_events):
        """n launches of the attention kernel of the self-attention call alone (operands already prepared in the
        set's own workspace), rotating over the input sets.  Returns the per-launch times in ms, or the mean
        over the whole loop when per_launch_events is false."""
        binding.regenvc_debug_set_phases(2 | KERNEL_BITS)
        try:
            if per_launch_events:
                evs = _events(n)
                for i, (a, b) in enumerate(evs):
                    s = sets[i % N_BUFFER_SETS]
                    binding.regenvc_set_workspace(s["ws"])
                    a.record(stream)
                    self_call(s)
                    b.record(stream)
                torch.cuda.synchronize()
                return [a.elapsed_time(b) for a, b in evs]
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(n):
                s = sets[i % N_BUFFER_SETS]
                binding.regenvc_set_workspace(s["ws"])
                self_call(s)
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n
        finally:
            binding.regenvc_set_workspace(None)
            binding.regenvc_debug_set_phases(3 | KERNEL_BITS)

    with torch.cuda.stream(stream):
        for i in range(max(args.warmup, 3)):
            step(sets[i % N_BUFFER_SETS])
        for s in sets:  # operands of every set prepared once in the set's own workspace (used by kernel_only_loop)
            binding.regenvc_set_workspace(s["ws"])
            self_call(s)
        binding.regenvc_set_workspace(None)

        # ---- the K timed steps of the contract
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        launches0 = binding.regenvc_kernel_launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            step(sets[i % N_BUFFER_SETS])
        e1.record(stream)
        barrier()
        sampler.stop()
        launches = binding.regenvc_kernel_launch_count() - launches0
        ms_total = e0.elapsed_time(e1)
        status = binding.regenvc_device_status(stream)
        if status != 0:
            raise SystemExit(f"device status {status}: {binding.status_string(status)}")

        # the same steps with the conditioning operands rewritten inside every cross-attention call, for comparison
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for i in range(args.steps):
            step_one_call_cross(sets[i % N_BUFFER_SETS])
        g1.record(stream)
        torch.cuda.synchronize()
        ms_step_one_call = g0.elapsed_time(g1) / args.steps

        # ---- the dominant kernel alone, burst regime: isolated launches right after a pause
        time.sleep(0.5)
        n_k = max(10, min(args.steps, 50))
        kernel_only_loop(3, True)
        burst_sampler = ClockSampler(local)
        burst_sampler.start()
        attn_times = kernel_only_loop(n_k, True)
        burst_sampler.stop()
        attn_ms, attn_ms_best = statistics.mean(attn_times), min(attn_times)
        binding.regenvc_debug_set_phases(1 | KERNEL_BITS)
        evp = _events(n_k)
        for i, (a, b) in enumerate(evp):
            a.record(stream)
            self_call(sets[i % N_BUFFER_SETS])
            b.record(stream)
        binding.regenvc_debug_set_phases(3 | KERNEL_BITS)
        torch.cuda.synchronize()
        prep_ms = statistics.mean(a.elapsed_time(b) for a, b in evp)

        # ---- sustained regime: the step loop repeated until at least --sustain-seconds have passed, whatever
        # --steps is, with the clocks sampled throughout; then the attention kernel alone in the same regime
        sustained = None
        if args.sustain_seconds > 0:
            chunk = max(8, int(0.05 / max(ms_total / args.steps * 1e-3, 1e-6)))  # about 50 ms of steps per event pair
            sus_sampler = ClockSampler(local)
            barrier()
            sus_sampler.start()
            t_wall0 = time.perf_counter()
            chunks, i = [], 0
            while True:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(chunk):
                    step(sets[i % N_BUFFER_SETS])
                    i += 1
                b.record(stream)
                chunks.append((a, b, time.perf_counter() - t_wall0))
                if len(chunks) >= 2:
                    chunks[-2][1].synchronize()  # keep one chunk queued behind the running one
                if time.perf_counter() - t_wall0 >= args.sustain_seconds and len(chunks) >= 4:
                    break
            torch.cuda.synchronize()
            t_wall = time.perf_counter() - t_wall0
            sus_sampler.stop()
            chunk_ms = [a.elapsed_time(b) / chunk for a, b, _ in chunks]
            settled = [m for m, (_, _, t) in zip(chunk_ms, chunks) if t >= 0.25 * t_wall] or chunk_ms
            # the kernel alone, still in the power-capped regime: about a second of back-to-back launches
            ker_sampler = ClockSampler(local)
            ker_sampler.start()
            n_sus_k = max(50, int(1.0 / max(attn_ms * 1e-3, 1e-6)))
            attn_ms_sus = kernel_only_loop(n_sus_k, False)
            ker_sampler.stop()
            sustained = {"seconds": t_wall, "steps": i, "ms_per_step": statistics.mean(settled),
                         "ms_per_step_all": statistics.mean(chunk_ms), "ms_per_step_first_chunk": chunk_ms[0],
                         "clocks": sus_sampler.summary(), "kernel_ms": attn_ms_sus, "kernel_launches": n_sus_k,
                         "kernel_clocks": ker_sampler.summary()}
            status = binding.regenvc_device_status(stream)
            if status != 0:
                raise SystemExit(f"device status {status}: {binding.status_string(status)}")

        # ---- producer fusion: the block's QKV projection with norm, rotation and operand layout fused into its
        # epilogue, followed by attention on those operands, against projection-then-attention (library GEMM and
        # element-wise kernels writing bf16 q, k, v, then the ordinary self-attention call)
        fusion = None
        if not args.no_producer and w.n_heads % 2 == 0:
            fusion = time_producer_fusion(binding, w, dev, stream)

        # ---- end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
        s0 = sets[0]
        e2e = None
        if not args.no_e2e:
            hq, hk, hv = (t.cpu().pin_memory() for t in (s0["q"], s0["k"], s0["v"]))
            hcross = [(a.cpu().pin_memory(), b.cpu().pin_memory()) for a, b in s0["cross"]]
            hout = torch.empty_like(hq).pin_memory()
            houtc = [torch.empty_like(hq).pin_memory() for _ in hcross]

            def host_step():
                binding.regenvc_attn_forward_host(hq, hk, hv, hout, w.T, w.H, w.W, w.theta, stream)
                for (ck, cv), oc in zip(hcross, houtc):
                    binding.regenvc_cross_attn_forward_host(hq, ck, cv, oc, stream)

            for _ in range(3):
                host_step()
            n_e = max(3, min(args.steps, 20))
            barrier()
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record(stream)
            for _ in range(n_e):
                host_step()
            f1.record(stream)
            barrier()
            e2e_ms = f0.elapsed_time(f1) / n_e
            qb = hq.numel() * 2
            h2d = 3 * qb + sum(qb + 2 * a.numel() * 2 for a, _ in hcross)
            d2h = qb * (1 + len(hcross))
            host0 = hout
            e2e = {"ms": e2e_ms, "h2d": h2d, "d2h": d2h, "steps": n_e}

    # max over ranks
    red = max_over_ranks([ms_total, e2e["ms"] if e2e else 0.0, attn_ms,
                          sustained["ms_per_step"] if sustained else 0.0,
                          sustained["kernel_ms"] if sustained else 0.0], dist, dev)
    ms_total, e2e_ms, attn_ms_max, sus_ms, sus_kernel_ms = red
    ms_step = ms_total / args.steps
    fl = step_flops(w)
    value = whole_job_tflops(world, fl, ms_step)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        burst_peak = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
        sus_peak = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
        achieved = w.self_flops() / (attn_ms * 1e-3) / 1e12
        bc = burst_sampler.summary()
        line = {
            "metric": "attention bf16 TFLOP/s", "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "fp16 operands (from bf16), fp32 accumulate, bf16 out",
            "data": "synthetic",
            "config": {"workload": w.name, "grid_THW": [w.T, w.H, w.W], "tokens": w.n_tokens, "heads": w.n_heads,
                       "head_dim": w.head_dim, "cross_kv": list(w.cross_kv), "layers": w.layers,
                       "denoise_steps": w.steps, "parallelism": f"{world} independent window(s), one per GPU",
                       "cross_attention": "on conditioning operands prepared once per sequence "
                                          "(regenvc_cross_kv_prepare, outside the timed steps)",
                       "communicator_ranks": ranks_seen,
                       "l2": f"{N_BUFFER_SETS} rotating input sets, each {4 * w.n_tokens * w.n_heads * 256 / 1e6:.0f} MB "
                             f"of q/k/v/out (L2 is 126 MB)"},
            "ms_per_window": ms_step * w.layers * w.steps,
            "ms_per_step_cross_prepared_in_call": ms_step_one_call,
            "pct_of_nominal_2250": 100.0 * value / world / NOMINAL_BF16_TFLOPS,
            "gpu_launches": int(launches),
            "clocks": sampler.summary(),
            # the kernel timed alone (isolated launches after a pause, rotating input sets) against the burst
            # figure of the measured cuBLAS bf16 peak: frac = achieved / peak, achieved = flops / kernel_ms_mean
            "roofline": {"bound": "tensor", "kernel": self_attention_kernel_name(w, torch.cuda.get_device_properties(dev).multi_processor_count),
                         "achieved": achieved, "peak": burst_peak, "unit": "TFLOP/s", "frac": achieved / burst_peak,
                         "peak_source": f"{peak_kind} cuBLAS bf16 burst (kernel timed alone; fp16 and bf16 operands "
                                        f"run at the same rate)",
                         "flops_per_launch": w.self_flops(),
                         "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                         "kernel_ms_mean": attn_ms, "kernel_ms_best": attn_ms_best, "kernel_launches_timed": n_k,
                         "kernel_sm_mhz_median": bc.get("sm_mhz"),
                         "kernel_time_x_mhz": attn_ms * bc["sm_mhz"] if bc.get("sm_mhz") else None,
                         "prep_kernel_ms": prep_ms,
                         "traffic": ATTN_KERNEL_DRAM_TRAFFIC_BYTES.get(w.name),
                         "algorithmic_hbm_bytes": 4.0 * w.n_tokens * w.n_heads * 256},
            "context": PAPER_CONTEXT,
        }
        if sustained:
            sc, kc = sustained["clocks"], sustained["kernel_clocks"]
            sus_tflops = whole_job_tflops(world, fl, sus_ms)
            sus_kernel_tflops = w.self_flops() / (sus_kernel_ms * 1e-3) / 1e12
            line["sustained"] = {
                "seconds": sustained["seconds"], "steps": sustained["steps"], "ms_per_step": sus_ms,
                "ms_per_step_whole_loop": sustained["ms_per_step_all"],
                "ms_per_step_first_chunk": sustained["ms_per_step_first_chunk"],
                "tflops": sus_tflops, "peak": sus_peak, "frac_of_sustained_peak": sus_tflops / world / sus_peak,
                "pct_of_nominal_2250": 100.0 * sus_tflops / world / NOMINAL_BF16_TFLOPS,
                "ms_per_window": sus_ms * w.layers * w.steps,
                "sm_mhz_median": sc.get("sm_mhz"), "power_w_max": sc.get("power_w_max"),
                "power_w_median": sc.get("power_w_median"), "clock_samples": sc.get("samples"),
                "reasons": sc.get("reasons"),
                "time_x_mhz": sus_ms * sc["sm_mhz"] if sc.get("sm_mhz") else None,
                "kernel": {"ms": sus_kernel_ms, "launches": sustained["kernel_launches"], "tflops": sus_kernel_tflops,
                           "frac_of_sustained_peak": sus_kernel_tflops / sus_peak,
                           "sm_mhz_median": kc.get("sm_mhz"), "clock_samples": kc.get("samples"),
                           "time_x_mhz": sus_kernel_ms * kc["sm_mhz"] if kc.get("sm_mhz") else None},
                "note": "step loop repeated for at least --sustain-seconds; ms_per_step is the mean after the "
                        "first quarter of the loop, max over ranks",
            }
        if fusion:
            line["producer_fusion"] = fusion
        if e2e:
            line["e2e"] = {"value": whole_job_tflops(world, fl, e2e_ms), "unit": "TFLOP/s",
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": e2e_ms, "steps": e2e["steps"]}
        if world == 1 and not args.no_cpu_baseline:
            import oracle

            oracle.build()
            heads = [0, w.n_heads // 2, w.n_heads - 1][: max(1, args.cpu_heads)]
            dt, flc = oracle_sample(w, heads, s0["q"].cpu(), s0["k"].cpu(), s0["v"].cpu(),
                                    [(a.cpu(), b.cpu()) for a, b in s0["cross"]])
            line["cpu_baseline"] = {"value": flc / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(),
                                    "kind": "oracle", "seconds": dt,
                                    "sample": f"heads {heads} of {w.n_heads}, all {w.n_tokens} query rows, self + cross"}
            # parity spot check of the timed configuration against the same oracle (first 8 rows, head 0)
            if host0 is not None:
                ref = oracle.self_attn_head(synth.bits(s0["q"].cpu()), synth.bits(s0["k"].cpu()),
                                            synth.bits(s0["v"].cpu()), w.T, w.H, w.W, 0, w.theta, rows=list(range(8)))
                got = host0[:8, 0].double().numpy()
                line["spot_check_mre"] = float(np.abs(got - ref).sum() / np.abs(ref).sum())
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------ Ulysses x Ring
def run_usp(args, w: synth.Workload):
    """--usp UxR: ONE window spread over U*R ranks the way the paper does it (Sec. 3.5): the token sequence is
    sharded over the ranks, an all-to-all inside each Ulysses group turns it into a head sharding, key/value
    blocks travel around the ring while the block-wise attention kernels run, and a second all-to-all restores
    the sequence sharding.  Strong scaling: the work of one window is fixed.  Rank 0 checks its own output shard
    against the oracle on sampled rows."""
    from paper_2607_28144_b200 import binding, build, usp

    build.build()
    U, R = (int(x) for x in args.usp.lower().split("x"))
    if U * R != args.gpus:
        raise SystemExit(f"--usp {args.usp} needs --gpus {U * R}")
    rank, world, local, dev, dist, ranks_seen = _setup_ranks(args)
    layout = usp.UspLayout(world, U, R, w.n_tokens, w.n_heads)
    pg_u = pg_r = None
    if world > 1:
        pg_u, pg_r = usp.make_groups(layout, rank, dist)
    q, k, v = synth.self_inputs(w)  # every rank draws the same window and keeps its own shard
    t0, cnt = layout.shard(rank)
    ql, kl, vl = (x[t0:t0 + cnt].contiguous().to(dev) for x in (q, k, v))
    attn = usp.UspAttention(layout, rank, pg_u, pg_r, ops=usp.CudaOps(), dist=dist)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    out = None
    for _ in range(max(args.warmup, 3)):
        out = attn(ql, kl, vl, w.T, w.H, w.W, w.theta)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = binding.regenvc_kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        out = attn(ql, kl, vl, w.T, w.H, w.W, w.theta)
    e1.record()
    barrier()
    sampler.stop()
    launches = binding.regenvc_kernel_launch_count() - launches0
    status = binding.regenvc_device_status()
    if status != 0:
        raise SystemExit(f"device status {status}: {binding.status_string(status)}")
    (ms_total,) = max_over_ranks([e0.elapsed_time(e1)], dist, dev)
    ms_step = ms_total / args.steps
    if rank == 0:
        line = {
            "metric": "attention bf16 TFLOP/s", "value": w.self_flops() / (ms_step * 1e-3) / 1e12, "unit": "TFLOP/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "fp16 operands (from bf16), fp32 accumulate, bf16 out", "data": "synthetic",
            "config": {"workload": w.name, "grid_THW": [w.T, w.H, w.W], "tokens": w.n_tokens, "heads": w.n_heads,
                       "head_dim": w.head_dim, "parallelism": f"one window over Ulysses {U} x Ring {R}",
                       "communicator_ranks": ranks_seen, "tokens_per_rank": cnt, "heads_per_rank": w.n_heads // U,
                       "note": "self-attention only; inputs and outputs stay sequence-sharded on the ranks"},
            "gpu_launches": int(launches), "clocks": sampler.summary(), "context": PAPER_CONTEXT,
        }
        if not args.no_cpu_baseline:
            import oracle

            oracle.build()
            rows = np.unique(np.concatenate([np.arange(min(4, cnt)), np.linspace(0, cnt - 1, num=min(24, cnt)).astype(np.int64)]))
            got = out.cpu()
            qb, kb, vb = synth.bits(q), synth.bits(k), synth.bits(v)
            num = den = 0.0
            for head in sorted({0, w.n_heads // 2, w.n_heads - 1}):
                ref = oracle.self_attn_head(qb, kb, vb, w.T, w.H, w.W, head, w.theta, rows=(rows + t0))
                num += float(np.abs(got[rows, head].double().numpy() - ref).sum())
                den += float(np.abs(ref).sum())
            line["shard_check_mre"] = num / den
            if num / den > 2e-3:
                raise SystemExit(f"rank 0's output shard disagrees with the oracle: mre {num / den}")
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def respawn_under_torchrun(args):
    """`python bench.py --gpus N` with N > 1 and no launcher: start the N ranks ourselves (one process per GPU,
    rendezvous on 127.0.0.1) by re-executing this command line under torch.distributed.run."""
    import socket

    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    os.execv(sys.executable, cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="window_480x832", choices=synth.WORKLOAD_ORDER)
    ap.add_argument("--usp", default=None, metavar="UxR",
                    help="spread ONE window over U*R = --gpus ranks as Ulysses x Ring (the paper's decomposition)")
    ap.add_argument("--sustain-seconds", type=float, default=4.0,
                    help="length of the sustained leg (the step loop repeated under the power cap); 0 skips it")
    ap.add_argument("--kernel", choices=["auto", "pair", "single"], default="auto",
                    help="auto: the library's own choice of self-attention kernel; pair / single: always the kernel "
                         "on pairs of thread blocks / always one thread block per work item (for profiles)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-producer", action="store_true", help="skip the producer-fusion leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-heads", type=int, default=3)
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        respawn_under_torchrun(args)
    if args.usp:
        run_usp(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
