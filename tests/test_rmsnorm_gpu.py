"""GPU parity of the RMSNorm QK-normalisation prologue (forward with tangent, backward through both outputs)
against the fp64 numpy oracle on the same seeded inputs, through the C-ABI binding.  Error metric per tensor:
max|gpu - ref| / max|ref|; bf16 mode 1e-2 (outputs are rounded to bf16 once; everything inside is fp32),
fp32 mode 1e-4.  The scale gradients are fp32 sums of fp32 terms over all B*H*N rows and are never rounded to
bf16: they are held to 1e-3 in bf16 mode and 1e-4 in fp32 mode.
"""
import numpy as np
import pytest
import torch

from oracle import qk_rmsnorm_numpy as orn
from paper_2511_19797_b200 import binding, inputs
from tests._parity import rel_err

pytestmark = pytest.mark.gpu


def _case(B, H, N, d, dtype, seed, eps):
    x = inputs.make_inputs(inputs.custom(B, H, N, d, seed=seed))
    g = torch.Generator(device="cpu")
    g.manual_seed(77 + seed)
    gQ = 1.0 + 0.3 * torch.randn(d, generator=g)
    gK = 1.0 + 0.3 * torch.randn(d, generator=g)
    # Q, tQ, K, tK and four cotangents (the other tensors of the recipe stand in for them)
    names = ("Q", "tQ", "K", "tK", "dO", "dtO", "V", "tV")
    t = {k: x[k].to(dtype) for k in names}
    dev = {k: v.cuda() for k, v in t.items()}
    f64 = {k: v.to(torch.float64).numpy() for k, v in t.items()}
    fw = binding.tvm_qk_rmsnorm_jvp_fwd(dev["Q"], dev["tQ"], dev["K"], dev["tK"], gQ.cuda(), gK.cuda(), eps=eps)
    bw = binding.tvm_qk_rmsnorm_jvp_bwd(dev["Q"], dev["tQ"], dev["K"], dev["tK"], gQ.cuda(), gK.cuda(), dev["dO"], dev["dtO"],
                                        dev["V"], dev["tV"], eps=eps)
    torch.cuda.synchronize()
    gq, gk = gQ.double().numpy(), gK.double().numpy()
    rQn, rtQn = orn.rmsnorm_jvp_fwd(f64["Q"], f64["tQ"], gq, eps)
    rKn, rtKn = orn.rmsnorm_jvp_fwd(f64["K"], f64["tK"], gk, eps)
    rdQ, rdtQ, rdgQ = orn.rmsnorm_jvp_bwd(f64["Q"], f64["tQ"], gq, f64["dO"], f64["dtO"], eps)
    rdK, rdtK, rdgK = orn.rmsnorm_jvp_bwd(f64["K"], f64["tK"], gk, f64["V"], f64["tV"], eps)
    ref = dict(Qn=rQn, tQn=rtQn, Kn=rKn, tKn=rtKn, dQ=rdQ, dtQ=rdtQ, dK=rdK, dtK=rdtK, dgQ=rdgQ, dgK=rdgK)
    got = dict(zip(("Qn", "tQn", "Kn", "tKn"), fw))
    got.update(zip(("dQ", "dtQ", "dK", "dtK", "dgQ", "dgK"), bw))
    return {k: rel_err(got[k].float().cpu().numpy(), ref[k]) for k in ref}


@pytest.mark.parametrize("B,H,N,d", [(2, 2, 64, 32), (1, 3, 257, 72), (2, 16, 1024, 72), (1, 2, 100, 64), (3, 1, 33, 128),
                                     (1, 1, 1, 8), (2, 5, 130, 40)])
@pytest.mark.parametrize("mode", ["bf16", "fp32"])
def test_rmsnorm_prologue_against_the_oracle(B, H, N, d, mode):
    dtype = torch.bfloat16 if mode == "bf16" else torch.float32
    errs = _case(B, H, N, d, dtype, seed=700 + N + d, eps=1e-6)
    tol = 1e-2 if mode == "bf16" else 1e-4
    tol_g = 1e-3 if mode == "bf16" else 1e-4
    bad = {k: e for k, e in errs.items() if not e <= (tol_g if k.startswith("dg") else tol)}
    assert not bad, (bad, errs)


def test_rmsnorm_prologue_with_a_large_epsilon():
    errs = _case(1, 2, 96, 48, torch.float32, seed=3, eps=0.5)
    assert max(errs.values()) <= 1e-4, errs


def test_rmsnorm_scale_gradients_are_bit_reproducible():
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(inputs.custom(2, 7, 333, 72, seed=5)).items()}
    g = torch.ones(72, device="cuda")
    runs = [binding.tvm_qk_rmsnorm_jvp_bwd(x["Q"], x["tQ"], x["K"], x["tK"], g, g, x["dO"], x["dtO"], x["V"], x["tV"]) for _ in range(2)]
    torch.cuda.synchronize()
    for a, b in zip(*runs):
        assert torch.equal(a, b)


def test_normalised_tensors_feed_the_attention():
    """The prologue's outputs are valid inputs of the attention forward (same layout, dtype and alignment)."""
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(inputs.custom(1, 2, 200, 72, seed=6)).items()}
    g = torch.ones(72, device="cuda")
    Qn, tQn, Kn, tKn = binding.tvm_qk_rmsnorm_jvp_fwd(x["Q"], x["tQ"], x["K"], x["tK"], g, g)
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(Qn, Kn, x["V"], tQn, tKn, x["tV"])
    binding.tvm_attn_check_status()
    assert torch.isfinite(O.float()).all() and torch.isfinite(tO.float()).all()
    # unit-RMS rows: |q . k| <= d, so the scaled scores are bounded by sqrt(d) and lse by log N + sqrt(d)
    assert float(lse.max()) <= np.log(200) + np.sqrt(72) + 1e-3
