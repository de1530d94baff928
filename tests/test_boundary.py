"""Host-side tests of the C ABI: the library loads without a GPU, exports every
symbol the header declares, and rejects bad arguments before any CUDA work."""
import ctypes
import os
import re

import pytest

from paper_2607_28144_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "regenvc_attn.h")


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def _declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(regenvc_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    declared = _declared_symbols()
    assert len(declared) >= 14
    for name in declared:
        assert hasattr(L, name), f"{name} declared in the header but not exported"
    assert sorted(binding.EXPORTS) == [d for d in declared if d in binding.EXPORTS]
    assert set(binding.EXPORTS) <= set(declared)


def test_status_strings_and_version(L):
    assert binding.regenvc_version().startswith("regenvc-attn")
    seen = {binding.status_string(c) for c in range(12)}
    assert len(seen) == 12 and binding.status_string(99) == "unknown status"


def test_workspace_bytes():
    # K' and V't, fp16, key count padded to 128, plus the fixed split-key scratch
    scratch = 160 * (256 * 128 * 4 + 256 * 8)
    assert scratch == 21_299_200
    assert binding.regenvc_workspace_bytes(10920, 12) == 2 * 12 * 11008 * 128 * 2 + scratch
    assert binding.regenvc_workspace_bytes(128, 2) == 2 * 2 * 128 * 128 * 2 + scratch
    assert binding.regenvc_workspace_bytes(1, 1) == 2 * 128 * 128 * 2 + scratch
    assert binding.regenvc_workspace_bytes(0, 1) == 0
    assert binding.regenvc_workspace_bytes(5, 1, 64) == 0


def test_argument_validation_happens_before_any_cuda_call(L):
    q, k, v, o = 0x10000, 0x20000, 0x30000, 0x40000  # never dereferenced: every call below must fail first
    f = L.regenvc_attn_forward
    assert f(None, k, v, o, 1, 1, 1, 1, 128, 1e4, None) == binding.ERR_NULL_POINTER
    assert f(q, k, v, None, 1, 1, 1, 1, 128, 1e4, None) == binding.ERR_NULL_POINTER
    assert f(q, k, v, o, 0, 1, 1, 1, 128, 1e4, None) == binding.ERR_BAD_SHAPE
    assert f(q, k, v, o, 1, -3, 1, 1, 128, 1e4, None) == binding.ERR_BAD_SHAPE
    assert f(q, k, v, o, 1, 1, 1, 0, 128, 1e4, None) == binding.ERR_BAD_SHAPE
    assert f(q, k, v, o, 2048, 2048, 2048, 1, 128, 1e4, None) == binding.ERR_BAD_SHAPE  # overflows
    assert f(q, k, v, o, 1, 1, 1, 1, 64, 1e4, None) == binding.ERR_UNSUPPORTED
    assert f(q + 8, k, v, o, 1, 1, 1, 1, 128, 1e4, None) == binding.ERR_MISALIGNED
    assert f(q, k, v, q + 128, 1, 1, 1, 1, 128, 1e4, None) == binding.ERR_ALIASING
    assert f(q, k, v, v, 1, 1, 1, 1, 128, 1e4, None) == binding.ERR_ALIASING
    assert f(q, k, v, o, 1, 1, 1, 1, 128, 0.0, None) == binding.ERR_UNSUPPORTED
    assert f(q, k, v, o, 1, 1, 1, 1, 128, float("nan"), None) == binding.ERR_UNSUPPORTED
    g = L.regenvc_cross_attn_forward
    assert g(q, None, v, o, 4, 4, 1, 128, None) == binding.ERR_NULL_POINTER
    assert g(q, k, v, o, 4, 0, 1, 128, None) == binding.ERR_BAD_SHAPE
    assert g(q, k, v, o, 4, 4, 1, 96, None) == binding.ERR_UNSUPPORTED
    assert g(q, k + 2, v, o, 4, 4, 1, 128, None) == binding.ERR_MISALIGNED
    assert g(q, k, v, k, 4, 4, 1, 128, None) == binding.ERR_ALIASING
    for host in (L.regenvc_attn_forward_host,):
        assert host(None, k, v, o, 1, 1, 1, 1, 128, 1e4, None) == binding.ERR_NULL_POINTER
        assert host(q, k, v, o, 1, 1, 1, 1, 32, 1e4, None) == binding.ERR_UNSUPPORTED
    assert L.regenvc_cross_attn_forward_host(q, k, v, q, 4, 4, 1, 128, None) == binding.ERR_ALIASING
    # the merge of partial results applies the same size limits as the calls that produce them
    ptrs = (ctypes.c_void_p * 2)(0x50000, 0x60000)
    m = L.regenvc_attn_merge
    assert m(ptrs, ptrs, 2, o, (1 << 30) + 1, 1, 128, None) == binding.ERR_BAD_SHAPE
    assert m(ptrs, ptrs, 2, o, 1 << 20, 1 << 11, 128, None) == binding.ERR_BAD_SHAPE   # n_q * n_heads = 2^31
    assert m(ptrs, ptrs, 2, o, 4, 70000, 128, None) == binding.ERR_BAD_SHAPE
    assert m(ptrs, ptrs, 9, o, 4, 1, 128, None) == binding.ERR_BAD_SHAPE
    assert m(ptrs, ptrs, 2, o, 4, 1, 64, None) == binding.ERR_UNSUPPORTED
    assert m(ptrs, ptrs, 2, None, 4, 1, 128, None) == binding.ERR_NULL_POINTER
    assert L.regenvc_static_device_status(None, None) == binding.ERR_NULL_POINTER
    assert L.regenvc_set_workspace(0x1001, 1 << 20) == binding.ERR_WORKSPACE
    assert L.regenvc_set_workspace(None, 0) == binding.OK
    assert L.regenvc_device_status(None, None) == binding.ERR_NULL_POINTER


def test_no_cpu_fallback_without_a_gpu(L):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    # valid arguments, but there is no device: the call must fail, never compute on the host
    buf = (ctypes.c_uint16 * (4 * 128))()
    a = ctypes.addressof(buf)
    a = (a + 15) & ~15
    rc = L.regenvc_cross_attn_forward(a, a + 256, a + 512, a + 768, 1, 1, 1, 128, None)
    assert rc in (binding.ERR_CUDA, binding.ERR_UNSUPPORTED)
    st = ctypes.c_int(0)
    assert L.regenvc_device_status(None, ctypes.byref(st)) in (binding.ERR_CUDA, binding.ERR_UNSUPPORTED)


def test_binding_rejects_cpu_tensors_for_device_entry_points():
    import torch

    t = torch.zeros((1, 1, 128), dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        binding.regenvc_attn_forward(t, t, t, t.clone(), 1, 1, 1)
    with pytest.raises(TypeError):
        binding.regenvc_cross_attn_forward(t, t, t, t.clone())
