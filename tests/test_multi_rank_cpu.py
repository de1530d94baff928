"""The N > 1 bookkeeping of bench.py on two gloo ranks (CPU): each rank gets its own window (distinct seeds),
times are reduced with MAX over ranks, and the whole-job rate counts every rank's window."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2607_28144_b200 import synth

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.WORKLOADS["tiny"]
        wi = synth.Workload(**{**w.__dict__, "seed": w.seed + bench.rank_seed_offset(0, rank)})
        q, _, _ = synth.self_inputs(wi)
        local_ms = [10.0 + 5.0 * rank, 3.0 - rank, 1.0]
        red = bench.max_over_ranks(local_ms, dist)
        gathered = [None] * world
        dist.all_gather_object(gathered, float(q.float().sum()))
        out[rank] = {"red": red, "sums": gathered,
                     "value": bench.whole_job_tflops(world, bench.step_flops(w), red[0])}
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_run_distinct_windows():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0]["red"] == out[1]["red"] == [15.0, 3.0, 1.0]
    assert out[0]["sums"] == out[1]["sums"] and out[0]["sums"][0] != out[0]["sums"][1]  # different windows
    import bench
    from paper_2607_28144_b200 import synth

    w = synth.WORKLOADS["tiny"]
    assert out[0]["value"] == pytest.approx(2 * bench.step_flops(w) / 15e-3 / 1e12)
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_bench_starts_its_own_ranks_and_fails_loudly_without_enough_gpus():
    """`python bench.py --gpus 2` without a launcher re-executes itself under torch.distributed.run (two ranks,
    rendezvous on 127.0.0.1).  On a machine with fewer than two GPUs every rank must stop with a clear message
    instead of quietly measuring one GPU."""
    import subprocess

    if torch.cuda.device_count() >= 2:
        pytest.skip("two GPUs are present: the command would run the benchmark itself")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1", "--warmup", "1"],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    text = r.stdout + r.stderr
    assert r.returncode != 0
    # (the launcher stops the other ranks as soon as the first one fails, so which rank's message gets out varies)
    assert "rank 1 needs cuda:1" in text or "rank 0 needs cuda:0" in text
    assert '"n_gpus"' not in r.stdout  # no result line
    # a rank count that contradicts --gpus is refused as well
    env2 = dict(env, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                       env=env2, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode != 0 and "WORLD_SIZE=1" in (r.stdout + r.stderr)
