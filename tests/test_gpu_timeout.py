"""The bounded waits of the kernels, exercised without faulting or hanging anything: a warp waits on a barrier
that nothing completes, gives up after its limit and records the timeout status; kernels that start while the
status is set skip their work; reading the status clears it and the next call is normal again."""
import time

import pytest
import torch

from paper_2607_28144_b200 import binding, synth
from parity_util import run_gpu_self

pytestmark = pytest.mark.gpu


def test_an_expired_wait_is_reported_and_cleared():
    assert binding.regenvc_device_status() == 0
    t0 = time.time()
    binding.regenvc_debug_expire_wait(500)
    assert binding.regenvc_device_status() == binding.ERR_TIMEOUT
    assert time.time() - t0 < 5.0           # the wait ended by itself, after about half a millisecond
    assert binding.regenvc_device_status() == 0   # cleared by the query
    assert binding.status_string(binding.ERR_TIMEOUT)
    with pytest.raises(binding.RegenvcError):
        binding.regenvc_debug_expire_wait(0)


def test_kernels_skip_their_work_while_the_status_is_set_and_recover_afterwards():
    w = synth.WORKLOADS["tiny"]
    q, k, v = synth.self_inputs(w)
    good = run_gpu_self(q, k, v, w.T, w.H, w.W)
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    out = torch.zeros_like(qd)
    binding.regenvc_debug_expire_wait(200)
    t0 = time.time()
    binding.regenvc_attn_forward(qd, kd, vd, out, w.T, w.H, w.W)   # starts with the status set: skips its work
    assert binding.regenvc_device_status() == binding.ERR_TIMEOUT    # the first error is kept
    assert time.time() - t0 < 5.0
    assert binding.regenvc_device_status() == 0
    again = run_gpu_self(q, k, v, w.T, w.H, w.W)
    assert torch.equal(again, good)
