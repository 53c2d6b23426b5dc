"""The allocation-free backward entry point, tvm_attn_jvp_bwd_noalloc, against tvm_attn_jvp_bwd.

Who needs it: callers that are handed tensors but may not allocate device memory where they call the
backward (a host framework with a fixed memory plan, a real-time loop, a plug-in without an allocator).
They cannot supply the workspace tvm_attn_jvp_bwd asks for, so the library keeps a fixed scratch array in
its own device image for them.  These tests call the entry point through the C ABI twice in a row (the
second call finds the array holding the first call's leftovers) and compare every gradient with the
workspace-taking entry point: both run the same kernels in the same order, so the results must be
bit-identical, which is well inside the tolerance of the other GPU parity tests.  One case sits exactly at
the size limit, one goes to the fp64 oracle, and one checks what the entry point exists for: that a call
leaves the amount of free device memory unchanged.  The file is collected last so that a run stopping at
the first failure has already run everything else.
"""
import ctypes

import pytest
import torch

from paper_2511_19797_b200 import binding, inputs
from tests._parity import assert_within, run_case

pytestmark = pytest.mark.gpu

NAMES = ("dQ", "dK", "dV", "dtQ", "dtK", "dtV")


def _setup(wl):
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()}
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"])
    args = (x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], O, tO, lse, mu, x["dO"], x["dtO"])
    return x, args


def _free_bytes():
    free, total = ctypes.c_size_t(0), ctypes.c_size_t(0)
    rt = ctypes.CDLL("libcudart.so.12")
    assert rt.cudaMemGetInfo(ctypes.byref(free), ctypes.byref(total)) == 0
    return free.value


@pytest.mark.parametrize("B,H,N,d", [(2, 2, 200, 72), (1, 3, 129, 64), (16, 16, 1024, 72)])
def test_noalloc_backward_matches_workspace_backward_twice(B, H, N, d):
    """The last shape has B*H*N = 262,144 rows: exactly TVM_ATTN_NOALLOC_MAX_ROWS, the whole scratch array in use."""
    assert B * H * N <= binding.NOALLOC_MAX_ROWS
    wl = inputs.custom(B, H, N, d, seed=31 + N)
    x, args = _setup(wl)
    ref = binding.tvm_attn_jvp_bwd(*args)
    binding.tvm_attn_check_status()
    for call in range(2):
        out = tuple(torch.full_like(x["Q"], float("nan")) for _ in range(6))  # allocated by the test, not the library
        got = binding.tvm_attn_jvp_bwd_noalloc(*args, out=out)
        binding.tvm_attn_check_status()
        for name, g, r in zip(NAMES, got, ref):
            assert torch.isfinite(g.float()).all(), (call, name)
            assert torch.equal(g, r), (call, name)


def test_noalloc_backward_against_the_oracle():
    errs, _, _ = run_case(inputs.custom(2, 3, 257, 72, seed=33), noalloc=True)
    assert_within(errs, 1e-2, 2e-2, 1e-4)


def test_noalloc_backward_allocates_no_device_memory():
    wl = inputs.custom(2, 4, 320, 72, seed=35)
    x, args = _setup(wl)
    out = tuple(torch.empty_like(x["Q"]) for _ in range(6))
    binding.tvm_attn_jvp_bwd_noalloc(*args, out=out)        # first call on this device: looks up the array's address
    torch.cuda.synchronize()
    try:
        free0 = _free_bytes()
    except OSError:
        pytest.skip("libcudart.so.12 not loadable by name")
    torch_alloc0, torch_reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    binding.tvm_attn_jvp_bwd_noalloc(*args, out=out)
    torch.cuda.synchronize()
    assert _free_bytes() >= free0, "the call took device memory"
    assert torch.cuda.memory_allocated() == torch_alloc0 and torch.cuda.memory_reserved() == torch_reserved0


def test_noalloc_backward_rejects_problems_beyond_its_scratch():
    lib = binding.load()
    rows = binding.NOALLOC_MAX_ROWS
    p = binding.Params(1, 1, rows + 8, 64, 0.0, binding.BF16, 0)   # B*H*N just over the limit
    ptrs = [ctypes.c_void_p(4096 + 16 * k) for k in range(18)]     # never dereferenced: the size check comes first
    assert lib.tvm_attn_jvp_bwd_noalloc(ctypes.byref(p), *ptrs, None) == -6
    assert b"NOALLOC" in lib.tvm_attn_strerror(-6)
