"""Helpers shared by the GPU parity tests: run the CUDA path through the C-ABI binding and the
C oracle on the same seeded inputs and report max|err| / max|ref| per output tensor."""
import numpy as np
import torch

from oracle import c_oracle
from paper_2511_19797_b200 import binding, inputs

FWD_NAMES = ("O", "tO", "lse", "mu")
BWD_NAMES = ("dQ", "dK", "dV", "dtQ", "dtK", "dtV")


def rel_err(got, ref):
    """max|got - ref| / max|ref|.  A reference that is identically zero (e.g. dQ when N = 1) has no
    scale of its own; its error is then reported in absolute terms (inputs are O(1))."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    if not np.all(np.isfinite(got)):
        return float("inf")
    scale = float(np.abs(ref).max())
    return float(np.abs(got - ref).max() / (scale if scale > 1e-12 else 1.0))


def run_case(wl, oracle_heads=None, dtype=torch.bfloat16, flags=0, scale=0.0, device="cuda:0", absent=None, noalloc=False):
    """Runs the whole workload on the GPU and the oracle on `oracle_heads` (flat b*H+h indices; all
    heads when None).  Returns ({name: rel_err}, gpu outputs, oracle outputs) over the compared heads.
    absent: "dO" or "dtO" -- that cotangent is passed to the library as a null pointer and to the oracle as zeros.
    noalloc: the backward goes through tvm_attn_jvp_bwd_noalloc (scratch inside the library)."""
    x = inputs.make_inputs(wl)
    if absent is not None:
        x[absent] = torch.zeros_like(x[absent])
    xr = {k: v.to(dtype) for k, v in x.items()}                      # what the GPU consumes
    B, H, N, d = xr["Q"].shape
    sel = None if oracle_heads is None else torch.as_tensor(list(oracle_heads), dtype=torch.long)

    def pick(t):  # (B,H,...) -> (heads,1,...)
        if sel is None:
            return t
        return t.reshape(B * H, 1, *t.shape[2:])[sel]

    xo = [pick(xr[k]).to(torch.float64).numpy() for k in inputs.NAMES]  # the same values, widened
    alpha = scale if scale else inputs.default_scale(d)
    dev = {k: v.to(device) for k, v in xr.items()}
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"],
                                              scale=scale, flags=flags)
    if noalloc:
        grads = binding.tvm_attn_jvp_bwd_noalloc(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], O, tO, lse, mu,
                                                 dev["dO"], dev["dtO"], out=tuple(torch.empty_like(O) for _ in range(6)),
                                                 scale=scale, flags=flags)
    else:
        grads = binding.tvm_attn_jvp_bwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], O, tO, lse, mu,
                                         None if absent == "dO" else dev["dO"], None if absent == "dtO" else dev["dtO"],
                                         scale=scale, flags=flags)
    binding.tvm_attn_check_status()
    got = dict(zip(FWD_NAMES + BWD_NAMES, [pick(t.float().cpu()).numpy() for t in (O, tO, lse, mu) + tuple(grads)]))
    rf = c_oracle.attn_jvp_fwd(*xo[:6], alpha)[:4]
    rb = c_oracle.attn_jvp_bwd(*xo, alpha)[:6]
    ref = dict(zip(FWD_NAMES + BWD_NAMES, rf + rb))
    errs = {k: rel_err(got[k], ref[k]) for k in ref}
    return errs, got, ref


def assert_within(errs, tol_fwd, tol_bwd, tol_stats=None):
    bad = {}
    for k, e in errs.items():
        tol = tol_fwd if k in ("O", "tO") else (tol_stats or tol_fwd) if k in ("lse", "mu") else tol_bwd
        if not e <= tol:
            bad[k] = (e, tol)
    assert not bad, "parity violated (err, tol): %r; all: %r" % (bad, errs)
