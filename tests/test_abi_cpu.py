"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every function the public
header declares, and its host-only entry points behave."""
import ctypes
import os
import re

import pytest

from paper_2511_19797_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "tvm_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tvm_(?:attn|qk)_[a-z_0-9]+)\s*\(", text)))


def test_header_functions_are_all_exported(lib):
    names = _declared_functions()
    assert {"tvm_attn_jvp_fwd", "tvm_attn_jvp_bwd", "tvm_attn_jvp_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), "library does not export %s" % n
    assert set(names) == set(binding.EXPORTS), "the binding's export list and the header disagree"


def test_version_and_strerror(lib):
    assert lib.tvm_attn_version() >= 100
    texts = [lib.tvm_attn_strerror(code) for code in (0, -1, -2, -3, -4, -5, -6)]
    assert all(len(t) > 0 for t in texts) and len(set(texts)) == len(texts)
    assert lib.tvm_attn_strerror(-99) == lib.tvm_attn_strerror(-1234)     # unknown codes share one text
    assert b"NOALLOC" in lib.tvm_attn_strerror(-6)


def test_noalloc_backward_rejects_problems_beyond_its_scratch_before_any_gpu_work(lib):
    rows = binding.NOALLOC_MAX_ROWS
    ptrs = [ctypes.c_void_p(4096 + 16 * k) for k in range(18)]     # never dereferenced: the size check comes first
    over = binding.Params(1, 1, rows + 8, 64, 0.0, binding.BF16, 0)
    assert lib.tvm_attn_jvp_bwd_noalloc(ctypes.byref(over), *ptrs, None) == -6
    over = binding.Params(16, 16, 1025, 72, 0.0, binding.BF16, 0)
    assert lib.tvm_attn_jvp_bwd_noalloc(ctypes.byref(over), *ptrs, None) == -6
    bad = binding.Params(1, 1, 64, 36, 0.0, binding.BF16, 0)
    assert lib.tvm_attn_jvp_bwd_noalloc(ctypes.byref(bad), *ptrs, None) == -2   # shape errors come first


def test_selftest_timeout_rejects_limits_out_of_range(lib):
    assert lib.tvm_attn_selftest_timeout(0, None) == -1
    assert lib.tvm_attn_selftest_timeout(10**9, None) == -1


def test_workspace_bytes_host_only():
    assert binding.tvm_attn_jvp_workspace_bytes(16, 16, 1024, 72, is_bwd=True) == 3 * 4 * 16 * 16 * 1024
    assert binding.tvm_attn_jvp_workspace_bytes(16, 16, 1024, 72, is_bwd=False) == 0
    # invalid parameters give 0
    assert binding.tvm_attn_jvp_workspace_bytes(0, 16, 1024, 72) == 0
    assert binding.tvm_attn_jvp_workspace_bytes(1, 1, 64, 132) == 0
    assert binding.tvm_attn_jvp_workspace_bytes(1, 1, 64, 36) == 0
    assert binding.tvm_attn_jvp_workspace_bytes(1, 1, 64, 32, dtype=7) == 0


def test_argument_errors_are_reported_before_any_gpu_work(lib):
    p = binding.Params(2, 2, 64, 32, 0.0, binding.BF16, 0)
    nul = [None] * 10
    assert lib.tvm_attn_jvp_fwd(ctypes.byref(p), *nul, None, 0, None) == -1      # null pointers
    assert lib.tvm_attn_jvp_fwd(None, *nul, None, 0, None) == -1                 # null params
    bad = binding.Params(2, 2, 64, 136, 0.0, binding.BF16, 0)
    assert lib.tvm_attn_jvp_fwd(ctypes.byref(bad), *nul, None, 0, None) == -2    # d > 128
    bad = binding.Params(2, 2, 64, 32, -1.0, binding.BF16, 0)
    assert lib.tvm_attn_jvp_fwd(ctypes.byref(bad), *nul, None, 0, None) == -1    # negative scale
    bad = binding.Params(2, 2, 64, 32, 0.0, binding.BF16, 8)
    assert lib.tvm_attn_jvp_bwd(ctypes.byref(bad), *([None] * 18), None, 0, None) == -1  # unknown flag
    ptrs = [ctypes.c_void_p(4096 + 16 * k) for k in range(18)]
    assert lib.tvm_attn_jvp_bwd(ctypes.byref(p), *ptrs, ctypes.c_void_p(8192), 16, None) == -3  # workspace too small
    ptrs[3] = ctypes.c_void_p(4100)
    assert lib.tvm_attn_jvp_bwd(ctypes.byref(p), *ptrs, ctypes.c_void_p(8192), 1 << 20, None) == -1  # misaligned


def test_binding_refuses_cpu_tensors():
    import torch
    x = torch.zeros(1, 1, 8, 8, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        binding.tvm_attn_jvp_fwd(x, x, x, x, x, x)
