"""GPU parity: the CUDA path, called through the C ABI binding, against the
fp64 oracle on the same seeded inputs (element by element on small shapes)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_28144_b200 import binding, synth
from parity_util import assert_parity, errors, f64, hull_check, run_gpu_cross, run_gpu_self

pytestmark = pytest.mark.gpu

D = 128


def _rand(rng, n, h, scale=1.0):
    return synth.from_f32(rng.standard_normal((n, h, D)) * scale)


def _self_case(T, H, W, h, seed, scale=1.0, theta=10000.0):
    rng = np.random.default_rng(seed)
    N = T * H * W
    q, k, v = _rand(rng, N, h, scale), _rand(rng, N, h, scale), _rand(rng, N, h, scale)
    gpu = f64(run_gpu_self(q, k, v, T, H, W, theta))
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W, theta)
    hull_check(gpu, f64(v))
    return assert_parity(gpu, ref, float(v.float().abs().max()), f"self {T}x{H}x{W} h={h}")


def test_workspace_holds_rotated_keys_and_transposed_values():
    """The preparation pass: K' equals the oracle's rotated keys to fp16 rounding; V't is V transposed exactly."""
    T, H, W, h = 3, 5, 11, 3
    N = T * H * W
    n_pad = (N + 127) // 128 * 128
    rng = np.random.default_rng(5)
    q, k, v = _rand(rng, N, h), _rand(rng, N, h), _rand(rng, N, h)
    nbytes = binding.regenvc_workspace_bytes(N, h)
    assert nbytes == 2 * h * n_pad * D * 2 + 21_299_200
    ws = torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda:0")
    binding.regenvc_set_workspace(ws)
    try:
        run_gpu_self(q, k, v, T, H, W)
    finally:
        binding.regenvc_set_workspace(None)
    halves = ws[: 2 * h * n_pad * D * 2].view(torch.float16).cpu()
    kp = halves[: h * n_pad * D].view(h, n_pad, D).double().numpy()
    vt = halves[h * n_pad * D:].view(h, D, n_pad).double().numpy()
    for a in range(h):
        ref = oracle.rope_rotate_head(synth.bits(k), T, H, W, a)
        np.testing.assert_allclose(kp[a, :N], ref, rtol=2 ** -10, atol=1e-6)
        assert (kp[a, N:] == 0).all() and (vt[a, :, N:] == 0).all()
        np.testing.assert_array_equal(vt[a, :, :N], f64(v)[:, a, :].T)


@pytest.mark.parametrize("grid,h", [
    ((1, 1, 1), 1), ((1, 1, 2), 1), ((2, 3, 4), 2), ((1, 1, 127), 1), ((1, 1, 129), 2), ((127, 1, 1), 1),
    ((1, 127, 1), 1), ((3, 5, 7), 3), ((2, 8, 8), 2), ((1, 11, 12), 1), ((1, 15, 17), 2), ((1, 16, 16), 3),
    ((1, 1, 257), 1), ((3, 7, 13), 2), ((2, 13, 17), 3), ((5, 9, 11), 2),
])
def test_self_attention_small_shapes(grid, h):
    T, H, W = grid
    _self_case(T, H, W, h, seed=1000 + T * H * W + h)


def test_self_attention_window_256x256():
    w = synth.WORKLOADS["window_256x256"]
    q, k, v = synth.self_inputs(w)
    gpu = f64(run_gpu_self(q, k, v, w.T, w.H, w.W, w.theta))
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), w.T, w.H, w.W, w.theta)
    hull_check(gpu, f64(v))
    e = assert_parity(gpu, ref, float(v.float().abs().max()), w.name)
    for a in range(w.n_heads):  # per head, to localise a bad head
        assert errors(gpu[:, a], ref[:, a], float(v.float().abs().max()))["mre"] <= 2e-3
    print("window_256x256", e)


@pytest.mark.parametrize("grid,h", [((7, 16, 16), 2), ((1, 25, 44), 3), ((2, 37, 29), 1), ((1, 40, 64), 5)])
def test_self_attention_with_split_key_pieces(grid, h):
    """Few work items and many key tiles: the library cuts the key range of every item into pieces (the
    incomplete-last-wave path) and merges the partial results; uneven pieces and a ragged last tile included."""
    T, H, W = grid
    _self_case(T, H, W, h, seed=4000 + T * H * W + h)


def test_cross_attention_with_split_key_pieces():
    rng = np.random.default_rng(4100)
    q, k, v = _rand(rng, 300, 2), _rand(rng, 1500, 2), _rand(rng, 1500, 2)
    gpu = f64(run_gpu_cross(q, k, v))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    assert_parity(gpu, ref, float(v.float().abs().max()), "cross 300x1500 split")


def test_tiny_workload_against_brute_force_too():
    w = synth.WORKLOADS["tiny"]
    q, k, v = synth.self_inputs(w)
    gpu = f64(run_gpu_self(q, k, v, w.T, w.H, w.W, w.theta))
    maxv = float(v.float().abs().max())
    for a in range(w.n_heads):
        assert_parity(gpu[:, a], oracle.brute_force(synth.bits(q), synth.bits(k), synth.bits(v), w.T, w.H, w.W, a),
                      maxv, "tiny vs brute force")
    assert_parity(gpu, oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), w.T, w.H, w.W), maxv, "tiny")


@pytest.mark.parametrize("scale", [0.5, 2.0])
def test_self_attention_score_range(scale):
    # q, k, v scaled: score standard deviation 0.25 and 4 (softmax from nearly flat to peaked)
    _self_case(2, 13, 17, 2, seed=77, scale=scale)


@pytest.mark.parametrize("theta", [1.0, 100.0, 1e6])
def test_self_attention_other_theta(theta):
    _self_case(3, 6, 9, 2, seed=78, theta=theta)


@pytest.mark.parametrize("n_q,n_kv,h", [
    (1, 1, 1), (1, 7, 2), (129, 127, 1), (129, 128, 2), (129, 129, 1), (1, 257, 2), (300, 257, 3), (1792, 512, 2),
    (129, 769, 2), (1792, 257, 12), (513, 512, 12),
])
def test_cross_attention(n_q, n_kv, h):
    rng = np.random.default_rng(2000 + n_q + n_kv + h)
    q, k, v = _rand(rng, n_q, h), _rand(rng, n_kv, h), _rand(rng, n_kv, h)
    gpu = f64(run_gpu_cross(q, k, v))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    hull_check(gpu, f64(v))
    assert_parity(gpu, ref, float(v.float().abs().max()), f"cross {n_q}x{n_kv} h={h}")


# ---------------------------------------------------------------- structured inputs that localise bugs
def test_zero_queries_give_column_mean_everywhere():
    T, H, W, h = 2, 11, 13, 2
    N = T * H * W
    rng = np.random.default_rng(31)
    k, v = _rand(rng, N, h), _rand(rng, N, h)
    q = torch.zeros_like(k)
    gpu = f64(run_gpu_self(q, k, v, T, H, W))
    mean = f64(v).mean(axis=0)
    assert np.abs(gpu - mean[None]).max() <= 2 ** -8 * np.abs(mean).max() + 1e-3


def test_constant_value_rows_come_back_exactly():
    T, H, W, h = 1, 9, 31, 2
    N = T * H * W
    rng = np.random.default_rng(32)
    q, k = _rand(rng, N, h, 2.0), _rand(rng, N, h, 2.0)
    crow = _rand(rng, 1, h)
    v = crow.expand(N, h, D).contiguous()
    gpu = f64(run_gpu_self(q, k, v, T, H, W))
    # sum_m p_m c / sum_m p_m = c up to fp32 accumulation and one bf16 rounding
    np.testing.assert_allclose(gpu, np.broadcast_to(f64(crow), gpu.shape), rtol=2 ** -8, atol=1e-6)


def test_position_probe_values():
    """v_m = (t, y, x, 1, m mod 128 one-hot ...): the output is the attention-weighted mean position and the
    probability mass per key residue; exposes a wrong token map, a dropped key tile or a wrong tail mask."""
    T, H, W, h = 3, 7, 15, 1
    N = T * H * W
    rng = np.random.default_rng(33)
    q, k = _rand(rng, N, h, 1.5), _rand(rng, N, h, 1.5)
    n = np.arange(N)
    v = np.zeros((N, h, D), dtype=np.float32)
    v[:, 0, 0], v[:, 0, 1], v[:, 0, 2], v[:, 0, 3] = n // (H * W), (n // W) % H, n % W, 1.0
    v[n, 0, 4 + (n % 124)] = 1.0
    v = synth.from_f32(v)
    gpu = f64(run_gpu_self(q, k, v, T, H, W))
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W)
    np.testing.assert_allclose(gpu[:, 0, 3], 1.0, rtol=2 ** -8)
    np.testing.assert_allclose(gpu[:, 0, 4:].sum(axis=1), 1.0, rtol=1e-2)
    assert_parity(gpu, ref, float(v.float().abs().max()), "position probe")


def test_dominating_key_and_large_scores():
    T, H, W, h = 1, 5, 60, 1
    N = T * H * W
    rng = np.random.default_rng(34)
    q, k, v = _rand(rng, N, h), _rand(rng, N, h), _rand(rng, N, h)
    gpu = f64(run_gpu_self(q, (k.float() * 6).to(torch.bfloat16), v, T, H, W))
    ref = oracle.self_attention(synth.bits(q), synth.bits((k.float() * 6).to(torch.bfloat16)), synth.bits(v), T, H, W)
    assert_parity(gpu, ref, float(v.float().abs().max()), "peaked softmax")


@pytest.mark.parametrize("growth", [3.0, 12.0, 40.0])
def test_scores_that_grow_along_the_sequence_force_reference_updates(growth):
    """Later key tiles hold much larger scores than the first one: the reference set on the first tile must be
    raised on the way (probabilities would leave the fp16 range otherwise), the accumulator rescaled and the
    tile redone (several times along the sequence for the larger growth factors)."""
    T, H, W, h = 1, 24, 50, 2
    N = T * H * W
    rng = np.random.default_rng(36)
    q, v = _rand(rng, N, h, 1.5), _rand(rng, N, h)
    ramp = (1.0 + (growth - 1.0) * np.arange(N) / (N - 1))[:, None, None]
    k = synth.from_f32(rng.standard_normal((N, h, D)) * ramp)
    gpu = f64(run_gpu_self(q, k, v, T, H, W))
    ref = oracle.self_attention(synth.bits(q), synth.bits(k), synth.bits(v), T, H, W)
    assert_parity(gpu, ref, float(v.float().abs().max()), f"growing scores x{growth}")


@pytest.mark.parametrize("amp", [3.5, 4.0, 5.0])
@pytest.mark.parametrize("key", [128 + 4, 128 + 13, 256 + 37, 128 + 0, 256 + 28])
def test_one_key_far_above_the_reference_of_the_earlier_tiles(key, amp):
    """Flat scores in the first key tile, then ONE key whose score lies 200 to 400 log2 units above them, placed
    both in columns whose exponential is evaluated by the polynomial (key index mod 16 in {4, 5}) and in
    MUFU columns: the jump must raise the reference (not wrap the polynomial's exponent field), so every output
    row equals that key's value vector."""
    n_q, n_kv, h = 200, 300, 2
    rng = np.random.default_rng(41)
    q = synth.from_f32(np.full((n_q, h, D), amp, dtype=np.float32))
    k = np.zeros((n_kv, h, D), dtype=np.float32)
    k[key] = amp                       # score 128 amp^2, times log2(e)/sqrt(128): 200 / 261 / 408 log2 units
    k = synth.from_f32(k)
    v = _rand(rng, n_kv, h)
    gpu = f64(run_gpu_cross(q, k, v))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    np.testing.assert_allclose(ref, np.broadcast_to(f64(v)[key], ref.shape), atol=1e-12)
    assert_parity(gpu, ref, float(v.float().abs().max()), f"jump at key {key}, amplitude {amp}")


@pytest.mark.parametrize("key", [900, 1290])
def test_a_saturation_in_one_work_item_only(key):
    """Eleven key tiles (the one-CTA-per-item kernel, not the persistent one), five work items per head.  The query
    rows 300..329 of head 0 and ONE late key point the same way with a score about 200 log2 units above everything
    else: the optimistic pass saturates in that work item alone, which is run again carefully (reference raised,
    accumulator rescaled) while every other item keeps the result of its clean first pass.  Those rows must equal
    the key's value vector, all others ordinary attention."""
    n_q, n_kv, h = 1100, 1300, 2
    rng = np.random.default_rng(43)
    q = rng.standard_normal((n_q, h, D)).astype(np.float32)
    k = rng.standard_normal((n_kv, h, D)).astype(np.float32)
    q[300:330, 0] = 3.5
    k[key, 0] = 3.5
    q, k, v = synth.from_f32(q), synth.from_f32(k), _rand(rng, n_kv, h)
    gpu = f64(run_gpu_cross(q, k, v))
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    np.testing.assert_allclose(ref[300:330, 0], np.broadcast_to(f64(v)[key, 0], (30, D)), atol=1e-9)
    assert_parity(gpu, ref, float(v.float().abs().max()), f"one saturating work item, key {key}")
    assert_parity(gpu[300:330, :1], ref[300:330, :1], float(v.float().abs().max()), "the saturated rows")


@pytest.mark.parametrize("b", [18.0, 20.5, 21.5, 23.0, 26.0])
@pytest.mark.parametrize("top_key", [5, 7000])
def test_one_dominating_key_over_a_flat_tail_of_twelve_thousand(b, top_key):
    """The worst case of the probabilities' fp16 floor: one key whose score lies `gap` log2 units above ALL the other
    12479 keys (gap = 8 b log2(e) / sqrt(128): 18.4 to 26.5), with values of opposite sign, so that whatever weight of
    the tail is lost shows up in full.  The kernels' softmax reference sits 4 log2 units above a row maximum: tail
    probabilities from about 21 log2 units below the largest one on vanish from P.V.  The result must stay within
    the stated error bound for every gap, wherever the dominating key comes (first tile or a late one)."""
    n_q, n_kv, h = 256, 12480, 1
    q = np.zeros((n_q, h, D), dtype=np.float32)
    k = np.zeros((n_kv, h, D), dtype=np.float32)
    v = -np.ones((n_kv, h, D), dtype=np.float32)
    q[:, 0, 0] = 8.0
    k[top_key, 0, 0] = b
    v[top_key] = 1.0
    rng = np.random.default_rng(71)
    q[:, 0, 1:] = 0.01 * rng.standard_normal((n_q, D - 1))   # (rows differ a little; these do not touch the scores' gap)
    q, k, v = synth.from_f32(q), synth.from_f32(k), synth.from_f32(v)
    ref = oracle.cross_attention(synth.bits(q), synth.bits(k), synth.bits(v))
    gap = 8.0 * b * np.log2(np.e) / np.sqrt(128.0)
    tail = (n_kv - 1) * 2.0 ** -gap
    np.testing.assert_allclose(ref[:, 0, 0], (1.0 - tail) / (1.0 + tail), rtol=1e-6)   # the oracle against the closed form
    for bits in (3, 3 | 8):
        binding.regenvc_debug_set_phases(bits)
        try:
            gpu = f64(run_gpu_cross(q, k, v))
        finally:
            binding.regenvc_debug_set_phases(3)
        err = np.abs(gpu - ref).max()
        assert err <= 1e-2, f"gap {gap:.1f} log2 units, kernel bits {bits}: max error {err:.2e} (tail weight {tail:.2e})"


def test_heads_are_independent_on_the_gpu():
    T, H, W, h = 2, 9, 10, 4
    N = T * H * W
    rng = np.random.default_rng(35)
    q, k, v = _rand(rng, N, h), _rand(rng, N, h), _rand(rng, N, h)
    full = run_gpu_self(q, k, v, T, H, W)
    sub = run_gpu_self(q[:, 1:3].contiguous(), k[:, 1:3].contiguous(), v[:, 1:3].contiguous(), T, H, W)
    assert torch.equal(full[:, 1:3], sub)


def test_repeated_calls_are_bitwise_reproducible_and_host_variant_matches():
    w = synth.WORKLOADS["tiny"]
    q, k, v = synth.self_inputs(w)
    a = run_gpu_self(q, k, v, w.T, w.H, w.W)
    b = run_gpu_self(q, k, v, w.T, w.H, w.W)
    assert torch.equal(a, b)
    out = torch.empty_like(q).pin_memory()
    binding.regenvc_attn_forward_host(q.pin_memory(), k.pin_memory(), v.pin_memory(), out, w.T, w.H, w.W)
    assert torch.equal(out, a)
    kc, vc = synth.cross_inputs(synth.WORKLOADS["window_480x832"], 257)
    kc, vc = kc[:, :2].contiguous(), vc[:, :2].contiguous()
    c = run_gpu_cross(q, kc, vc)
    outc = torch.empty_like(q)
    binding.regenvc_cross_attn_forward_host(q, kc, vc, outc)
    assert torch.equal(outc, c)


def test_out_of_range_input_sets_the_range_status():
    q = torch.zeros((4, 1, D), dtype=torch.bfloat16)
    k = torch.zeros((4, 1, D), dtype=torch.bfloat16)
    k[2, 0, 5] = 1e6  # beyond fp16
    dev = torch.device("cuda:0")
    out = torch.empty((4, 1, D), dtype=torch.bfloat16, device=dev)
    binding.regenvc_cross_attn_forward(q.to(dev), k.to(dev), k.to(dev), out)
    assert binding.regenvc_device_status() == binding.ERR_RANGE
    assert binding.regenvc_device_status() == 0  # cleared by the query


def test_workspace_too_small_is_rejected():
    dev = torch.device("cuda:0")
    t = torch.zeros((200, 1, D), dtype=torch.bfloat16, device=dev)
    ws = torch.empty((1024,), dtype=torch.uint8, device=dev)
    binding.regenvc_set_workspace(ws)
    try:
        with pytest.raises(binding.RegenvcError) as ei:
            binding.regenvc_cross_attn_forward(t, t, t, torch.empty_like(t))
        assert ei.value.code == binding.ERR_WORKSPACE
    finally:
        binding.regenvc_set_workspace(None)


def test_warm_calls_can_be_captured_in_a_cuda_graph_and_replayed():
    """A warm call allocates nothing and never synchronises, so a whole step (self-attention plus cross-attention)
    can be recorded once and replayed; the replay on new input values must equal direct calls bit for bit."""
    w = synth.WORKLOADS["window_256x256"]
    dev = torch.device("cuda:0")
    q, k, v = (t.to(dev) for t in synth.self_inputs(w))
    kc, vc = (t[:, : w.n_heads].contiguous().to(dev) for t in synth.cross_inputs(synth.WORKLOADS["window_480x832"], 512))
    out_s, out_c = torch.empty_like(q), torch.empty_like(q)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(2):  # warm-up on the capturing stream: workspace, tables, kernel attributes
            binding.regenvc_attn_forward(q, k, v, out_s, w.T, w.H, w.W)
            binding.regenvc_cross_attn_forward(q, kc, vc, out_c)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        binding.regenvc_attn_forward(q, k, v, out_s, w.T, w.H, w.W)
        binding.regenvc_cross_attn_forward(q, kc, vc, out_c)
    # new values in the same buffers, then replay
    w2 = synth.Workload(**{**w.__dict__, "seed": w.seed + 1000})
    q2, k2, v2 = synth.self_inputs(w2)
    q.copy_(q2.to(dev)); k.copy_(k2.to(dev)); v.copy_(v2.to(dev))
    out_s.zero_(); out_c.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert binding.regenvc_device_status() == 0
    ref_s, ref_c = torch.empty_like(q), torch.empty_like(q)
    binding.regenvc_attn_forward(q, k, v, ref_s, w.T, w.H, w.W)
    binding.regenvc_cross_attn_forward(q, kc, vc, ref_c)
    torch.cuda.synchronize()
    assert torch.equal(out_s, ref_s) and torch.equal(out_c, ref_c)
    assert float(out_s.float().abs().max()) > 0


def test_two_host_threads_on_their_own_streams_do_not_disturb_each_other():
    """The internal workspace is per host thread, so calls from two threads may overlap on the GPU."""
    import threading

    w = synth.WORKLOADS["window_256x256"]
    dev = torch.device("cuda:0")
    inputs = []
    for i in range(2):
        wi = synth.Workload(**{**w.__dict__, "seed": w.seed + 50 + i})
        inputs.append([t.to(dev) for t in synth.self_inputs(wi)])
    want = []
    for q, k, v in inputs:
        o = torch.empty_like(q)
        binding.regenvc_attn_forward(q, k, v, o, w.T, w.H, w.W)
        want.append(o)
    torch.cuda.synchronize()
    got = [[None] * 6 for _ in range(2)]
    errors_seen = []

    def work(i):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            q, k, v = inputs[i]
            with torch.cuda.stream(stream):
                for r in range(6):
                    o = torch.empty_like(q)
                    binding.regenvc_attn_forward(q, k, v, o, w.T, w.H, w.W, stream=stream)
                    got[i][r] = o
            stream.synchronize()
        except Exception as e:  # pragma: no cover
            errors_seen.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors_seen, errors_seen
    torch.cuda.synchronize()
    assert binding.regenvc_device_status() == 0
    for i in range(2):
        for r in range(6):
            assert torch.equal(got[i][r], want[i]), f"thread {i} call {r}"


def test_one_thread_two_streams_share_the_default_workspace_safely():
    """A self-attention call on one stream and a cross-attention call on another, both from this thread, use the
    same default workspace: the library orders the second behind the first on the GPU, so both results equal
    those of the same calls made one after the other."""
    w = synth.WORKLOADS["window_256x256"]
    dev = torch.device("cuda:0")
    q, k, v = (t.to(dev) for t in synth.self_inputs(w))
    kc, vc = (t[:, : w.n_heads].contiguous().to(dev) for t in synth.cross_inputs(synth.WORKLOADS["window_480x832"], 512))
    want_s, want_c = torch.empty_like(q), torch.empty_like(q)
    binding.regenvc_attn_forward(q, k, v, want_s, w.T, w.H, w.W)
    binding.regenvc_cross_attn_forward(q, kc, vc, want_c)
    torch.cuda.synchronize()
    a, b = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(20):
        got_s, got_c = torch.full_like(q, float("nan")), torch.full_like(q, float("nan"))
        torch.cuda.synchronize()
        binding.regenvc_attn_forward(q, k, v, got_s, w.T, w.H, w.W, stream=a)
        binding.regenvc_cross_attn_forward(q, kc, vc, got_c, stream=b)
        binding.regenvc_attn_forward(q, k, v, got_s, w.T, w.H, w.W, stream=a)
        torch.cuda.synchronize()
        assert torch.equal(got_s, want_s) and torch.equal(got_c, want_c)
    assert binding.regenvc_device_status() == 0
