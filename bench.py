#!/usr/bin/env python
"""Benchmark of the fused 3D-RoPE attention path on seeded synthetic tensors.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the whole hot path over one window: the
self-attention call (key/value preparation pass + attention kernel) followed by
one cross-attention call per conditioning sequence of the workload.  At N = 1
the workload is the 480x832 window (7x30x52 = 10920 tokens, 12 heads x 128,
plus 512 conditioning tokens), the shape the tensor-peak target is quoted on.
With N > 1 (one process per GPU under torchrun) every rank runs its own window
(heads and windows are independent: no data-path collective, weak scaling).

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
# shape, from the ncu capture summarised in profiles/attn_pipelined_kernel_window_480x832.md (101.5 MB + 18.0 MB).
ATTN_KERNEL_DRAM_TRAFFIC_BYTES = {"window_480x832": 119.4e6}
N_BUFFER_SETS = 4


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
            time.sleep(0.005)

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
                "power_w_max": max(self.power) if self.power else None}


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
def run_ours(args, w: synth.Workload):
    from paper_2607_28144_b200 import binding, build

    build.build()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)

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
                     "out": torch.empty_like(q, device=dev), "outc": [torch.empty_like(q, device=dev) for _ in cross]})
    host0 = None
    stream = torch.cuda.Stream(device=dev)

    def step(s):
        binding.regenvc_attn_forward(s["q"], s["k"], s["v"], s["out"], w.T, w.H, w.W, w.theta, stream)
        for (ck, cv), oc in zip(s["cross"], s["outc"]):
            binding.regenvc_cross_attn_forward(s["q"], ck, cv, oc, stream)

    with torch.cuda.stream(stream):
        for i in range(max(args.warmup, 3)):
            step(sets[i % N_BUFFER_SETS])
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

        # the dominant kernel alone: attention kernel of the self-attention call (operands already prepared)
        s0 = sets[0]
        step(s0)
        binding.regenvc_attn_forward(s0["q"], s0["k"], s0["v"], s0["out"], w.T, w.H, w.W, w.theta, stream)
        binding.regenvc_debug_set_phases(2)
        n_k = max(10, min(args.steps, 50))
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_k)]
        for a, b in evs:
            a.record(stream)
            binding.regenvc_attn_forward(s0["q"], s0["k"], s0["v"], s0["out"], w.T, w.H, w.W, w.theta, stream)
            b.record(stream)
        binding.regenvc_debug_set_phases(1)
        evp = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_k)]
        for a, b in evp:
            a.record(stream)
            binding.regenvc_attn_forward(s0["q"], s0["k"], s0["v"], s0["out"], w.T, w.H, w.W, w.theta, stream)
            b.record(stream)
        binding.regenvc_debug_set_phases(3)
        torch.cuda.synchronize()
        attn_ms = statistics.mean(a.elapsed_time(b) for a, b in evs)
        attn_ms_best = min(a.elapsed_time(b) for a, b in evs)
        prep_ms = statistics.mean(a.elapsed_time(b) for a, b in evp)

        # end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
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
            t0 = time.perf_counter()
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
    ms_total, e2e_ms, attn_ms_max = max_over_ranks([ms_total, e2e["ms"] if e2e else 0.0, attn_ms], dist, dev)
    ms_step = ms_total / args.steps
    fl = step_flops(w)
    value = whole_job_tflops(world, fl, ms_step)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        peak = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
        achieved = w.self_flops() / (attn_ms * 1e-3) / 1e12
        line = {
            "metric": "attention bf16 TFLOP/s", "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "fp16 operands (from bf16), fp32 accumulate, bf16 out",
            "data": "synthetic",
            "config": {"workload": w.name, "grid_THW": [w.T, w.H, w.W], "tokens": w.n_tokens, "heads": w.n_heads,
                       "head_dim": w.head_dim, "cross_kv": list(w.cross_kv), "layers": w.layers,
                       "denoise_steps": w.steps, "parallelism": f"{world} independent window(s), one per GPU",
                       "l2": f"{N_BUFFER_SETS} rotating input sets, each {4 * w.n_tokens * w.n_heads * 256 / 1e6:.0f} MB "
                             f"of q/k/v/out (L2 is 126 MB)"},
            "ms_per_window": ms_step * w.layers * w.steps,
            "pct_of_nominal_2250": 100.0 * value / world / NOMINAL_BF16_TFLOPS,
            "gpu_launches": int(launches),
            "clocks": sampler.summary(),
            "roofline": {"bound": "tensor", "kernel": "attn_pipelined_kernel (self-attention)",
                         "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_source": f"{peak_kind} cuBLAS bf16 sustained (kernel timed in a back-to-back loop; "
                                        f"fp16 and bf16 operands run at the same rate)",
                         "frac_of_burst": achieved / float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])),
                         "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                         "kernel_ms_mean": attn_ms, "kernel_ms_best": attn_ms_best, "prep_kernel_ms": prep_ms,
                         "traffic": ATTN_KERNEL_DRAM_TRAFFIC_BYTES.get(w.name),
                         "algorithmic_hbm_bytes": 4.0 * w.n_tokens * w.n_heads * 256},
            "context": PAPER_CONTEXT,
        }
        if e2e:
            line["e2e"] = {"value": whole_job_tflops(world, fl, e2e_ms), "unit": "TFLOP/s",
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": e2e_ms, "steps": e2e["steps"]}
        if world == 1 and not args.no_cpu_baseline:
            import oracle

            oracle.build()
            s0 = sets[0]
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="window_480x832", choices=synth.WORKLOAD_ORDER)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-heads", type=int, default=3)
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
