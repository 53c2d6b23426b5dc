"""The allocation-free backward entry point, tvm_attn_jvp_bwd_noalloc, against tvm_attn_jvp_bwd.

Who needs it: callers that are handed tensors but may not allocate device memory where they call the
backward (a host framework with a fixed memory plan, a real-time loop, a plug-in without an allocator).
They cannot supply the workspace tvm_attn_jvp_bwd asks for, so the library keeps a fixed scratch array in
its own device image for them.  This test calls the entry point through the C ABI twice in a row (the
second call finds the array holding the first call's leftovers) and compares every gradient with the
workspace-taking entry point, within the tolerance of the other GPU parity tests.  It is collected last so
that a run stopping at the first failure has already run everything else.
"""
import ctypes

import pytest
import torch

from paper_2511_19797_b200 import binding, inputs

pytestmark = pytest.mark.gpu

BF16_BWD = 2e-2  # max|a - b| / max|b|, as in test_parity_gpu.py


def _setup(wl):
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()}
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"])
    args = (x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], O, tO, lse, mu, x["dO"], x["dtO"])
    return x, args


@pytest.mark.parametrize("B,H,N,d", [(2, 2, 200, 72), (1, 3, 129, 64)])
def test_noalloc_backward_matches_workspace_backward_twice(B, H, N, d):
    wl = inputs.custom(B, H, N, d, seed=31 + N)
    x, args = _setup(wl)
    ref = binding.tvm_attn_jvp_bwd(*args)
    binding.tvm_attn_check_status()
    for call in range(2):
        out = tuple(torch.full_like(x["Q"], float("nan")) for _ in range(6))  # allocated by the test, not the library
        got = binding.tvm_attn_jvp_bwd_noalloc(*args, out=out)
        binding.tvm_attn_check_status()
        for name, g, r in zip(("dQ", "dK", "dV", "dtQ", "dtK", "dtV"), got, ref):
            g32, r32 = g.float(), r.float()
            assert torch.isfinite(g32).all(), (call, name)
            err = float((g32 - r32).abs().max() / r32.abs().max().clamp_min(1e-12))
            assert err <= BF16_BWD, (call, name, err)


def test_noalloc_backward_rejects_problems_beyond_its_scratch():
    lib = binding.load()
    rows = binding.NOALLOC_MAX_ROWS
    p = binding.Params(1, 1, rows + 8, 64, 0.0, binding.BF16, 0)   # B*H*N just over the limit
    ptrs = [ctypes.c_void_p(4096 + 16 * k) for k in range(18)]     # never dereferenced: the size check comes first
    assert lib.tvm_attn_jvp_bwd_noalloc(ctypes.byref(p), *ptrs, None) == -6
    assert b"NOALLOC" in lib.tvm_attn_strerror(-6)
