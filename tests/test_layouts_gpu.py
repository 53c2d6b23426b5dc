"""Shape generality of the attention-JVP path on the GPU: M queries against N keys (App. C "Background":
Q in R^{M x d}, K, V in R^{N x d}) and tensors read and written in place with row / head / batch strides, e.g. the
(B, rows, H, d) layout of a transformer block or the Q, K, V slices of a fused projection.

M != N is compared with the whole-matrix numpy oracle (it takes different numbers of query and key rows) at the
tolerances of the other parity tests.  A strided call runs the same kernels in the same order as the packed call
on the same values, so its results must be bit-identical to the packed ones; one strided case also goes to the
oracle directly.
"""
import numpy as np
import pytest
import torch

from oracle import attn_jvp_numpy as onp
from paper_2511_19797_b200 import binding, inputs
from tests._parity import BWD_NAMES, FWD_NAMES, assert_within, rel_err

pytestmark = pytest.mark.gpu

Q_SIDE = ("Q", "tQ", "dO", "dtO")
K_SIDE = ("K", "V", "tK", "tV")


def _draw(B, H, M, N, d, seed, dtype):
    """The eight tensors of the recipe, the query-side ones cut to M rows and the key-side ones to N rows."""
    x = inputs.make_inputs(inputs.custom(B, H, max(M, N), d, seed=seed))
    out = {}
    for k in Q_SIDE:
        out[k] = x[k][:, :, :M].contiguous().to(dtype)
    for k in K_SIDE:
        out[k] = x[k][:, :, :N].contiguous().to(dtype)
    return out


def _gpu(dev, flags=0):
    fw = binding.tvm_attn_jvp_fwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], flags=flags)
    gr = binding.tvm_attn_jvp_bwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], *fw, dev["dO"], dev["dtO"],
                                  flags=flags)
    binding.tvm_attn_check_status()
    return dict(zip(FWD_NAMES + BWD_NAMES, tuple(fw) + tuple(gr)))


def _oracle(x, d):
    f = {k: v.to(torch.float64).numpy() for k, v in x.items()}
    alpha = inputs.default_scale(d)
    rf = onp.attn_jvp_fwd(f["Q"], f["K"], f["V"], f["tQ"], f["tK"], f["tV"], alpha)
    rb = onp.attn_jvp_bwd(f["Q"], f["K"], f["V"], f["tQ"], f["tK"], f["tV"], f["dO"], f["dtO"], alpha)
    return dict(zip(FWD_NAMES + BWD_NAMES, tuple(rf) + tuple(rb)))


@pytest.mark.parametrize("B,H,M,N,d", [(2, 3, 100, 260, 72), (1, 2, 300, 64, 64), (1, 4, 1, 130, 40), (2, 2, 129, 1, 80),
                                       (1, 2, 640, 77, 72), (2, 40, 65, 200, 72), (1, 1, 77, 1000, 24)])
@pytest.mark.parametrize("mode", ["bf16", "fp32"])
def test_cross_attention_against_the_oracle(B, H, M, N, d, mode):
    dtype = torch.bfloat16 if mode == "bf16" else torch.float32
    x = _draw(B, H, M, N, d, seed=900 + M + N, dtype=dtype)
    got = _gpu({k: v.cuda() for k, v in x.items()})
    ref = _oracle(x, d)
    assert tuple(got["O"].shape) == (B, H, M, d) and tuple(got["dK"].shape) == (B, H, N, d) and tuple(got["lse"].shape) == (B, H, M)
    errs = {k: rel_err(got[k].float().cpu().numpy(), ref[k]) for k in ref}
    if mode == "bf16":
        assert_within(errs, 1e-2, 2e-2, 1e-4)
    else:
        assert_within(errs, 1e-4, 1e-4)


def _as_bnhd(t):
    """The same values stored (B, rows, H, d), viewed (B, H, rows, d): row stride H*d, head stride d."""
    return t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)


@pytest.mark.parametrize("B,H,M,N,d", [(2, 3, 200, 200, 72), (1, 5, 129, 129, 64), (2, 4, 100, 260, 72), (3, 50, 192, 192, 72)])
@pytest.mark.parametrize("flags", [0, binding.FLAG_CUDA_CORES])
def test_token_major_layout_gives_the_packed_results_bit_for_bit(B, H, M, N, d, flags):
    x = _draw(B, H, M, N, d, seed=40 + M, dtype=torch.bfloat16)
    dev = {k: v.cuda() for k, v in x.items()}
    packed = _gpu(dev, flags)
    strided = _gpu({k: _as_bnhd(v) for k, v in dev.items()}, flags)
    for k in packed:
        if k not in ("lse", "mu"):
            assert strided[k].stride() != packed[k].stride() or H == 1, k
        assert torch.equal(strided[k], packed[k]), k


def test_fused_qkv_projection_buffers_in_place():
    """Q, K, V (and their tangents, and the gradients) as slices of (B, N, 3, H, d) buffers, as a fused projection
    leaves them: nothing is copied, nothing outside the slices is written, results equal the packed call's."""
    B, H, N, d = 2, 6, 200, 72
    x = _draw(B, H, N, N, d, seed=51, dtype=torch.bfloat16)
    dev = {k: v.cuda() for k, v in x.items()}
    packed = _gpu(dev)

    def fused(q, k, v):
        buf = torch.full((B, N, 4, H, d), 9.0, dtype=torch.bfloat16, device="cuda")   # slot 3: a canary
        for i, t in enumerate((q, k, v)):
            buf[:, :, i] = t.permute(0, 2, 1, 3)
        return buf, [buf[:, :, i].permute(0, 2, 1, 3) for i in range(3)]

    pbuf, (Q, K, V) = fused(dev["Q"], dev["K"], dev["V"])
    tbuf, (tQ, tK, tV) = fused(dev["tQ"], dev["tK"], dev["tV"])
    gbuf = torch.full((B, N, 4, H, d), 9.0, dtype=torch.bfloat16, device="cuda")
    tgbuf = torch.full_like(gbuf, 9.0)
    dQ, dK, dV = (gbuf[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    dtQ, dtK, dtV = (tgbuf[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    cot = {k: _as_bnhd(dev[k]) for k in ("dO", "dtO")}
    assert not Q.is_contiguous() and Q.stride() == (N * 4 * H * d, d, 4 * H * d, 1)
    # outputs of the forward in the token-major layout of the cotangents (all query-side tensors share one layout)
    O = torch.empty_strided(cot["dO"].shape, cot["dO"].stride(), dtype=torch.bfloat16, device="cuda")
    tO = torch.empty_strided(cot["dO"].shape, cot["dO"].stride(), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ValueError):       # Q (stride 4*H*d) and O (stride H*d) are both query-side: layouts must agree
        binding.tvm_attn_jvp_fwd(Q, K, V, tQ, tK, tV, out=(O, tO, torch.empty(B, H, N, device="cuda"), torch.empty(B, H, N, device="cuda")))
    # so the query side lives in its own (B, N, 1+..) buffers with the fused stride: O, tO, dO, dtO in (B, N, 4, H, d) too
    obuf = torch.full((B, N, 4, H, d), 9.0, dtype=torch.bfloat16, device="cuda")
    O, tO = obuf[:, :, 0].permute(0, 2, 1, 3), obuf[:, :, 1].permute(0, 2, 1, 3)
    cbuf = torch.full((B, N, 4, H, d), 9.0, dtype=torch.bfloat16, device="cuda")
    cbuf[:, :, 0] = dev["dO"].permute(0, 2, 1, 3)
    cbuf[:, :, 1] = dev["dtO"].permute(0, 2, 1, 3)
    G, Hc = cbuf[:, :, 0].permute(0, 2, 1, 3), cbuf[:, :, 1].permute(0, 2, 1, 3)
    lse, mu = torch.empty(B, H, N, device="cuda"), torch.empty(B, H, N, device="cuda")
    binding.tvm_attn_jvp_fwd(Q, K, V, tQ, tK, tV, out=(O, tO, lse, mu))
    binding.tvm_attn_jvp_bwd(Q, K, V, tQ, tK, tV, O, tO, lse, mu, G, Hc, out=(dQ, dK, dV, dtQ, dtK, dtV))
    binding.tvm_attn_check_status()
    got = dict(O=O, tO=tO, lse=lse, mu=mu, dQ=dQ, dK=dK, dV=dV, dtQ=dtQ, dtK=dtK, dtV=dtV)
    for k, v in got.items():
        assert torch.equal(v, packed[k]), k
    for buf in (gbuf, tgbuf):
        assert torch.all(buf[:, :, 3] == 9.0), "wrote outside the gradient slices"
    assert torch.all(obuf[:, :, 2:] == 9.0) and torch.all(pbuf[:, :, 3] == 9.0) and torch.all(tbuf[:, :, 3] == 9.0)


def test_strided_cross_attention_against_the_oracle():
    B, H, M, N, d = 2, 3, 150, 333, 72
    x = _draw(B, H, M, N, d, seed=61, dtype=torch.bfloat16)
    got = _gpu({k: _as_bnhd(v.cuda()) for k, v in x.items()})
    ref = _oracle(x, d)
    errs = {k: rel_err(got[k].float().cpu().numpy(), ref[k]) for k in ref}
    assert_within(errs, 1e-2, 2e-2, 1e-4)


def test_detached_backward_in_the_token_major_layout():
    """Absent dtO with strided outputs: the tangent gradients that are given come back zero, row by row."""
    B, H, N, d = 2, 3, 130, 72
    x = _draw(B, H, N, N, d, seed=71, dtype=torch.bfloat16)
    dev = {k: _as_bnhd(v.cuda()) for k, v in x.items()}
    fw = binding.tvm_attn_jvp_fwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"])
    outs = tuple(torch.full((B, N, H, d), 5.0, dtype=torch.bfloat16, device="cuda").permute(0, 2, 1, 3) for _ in range(6))
    binding.tvm_attn_jvp_bwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], *fw, dev["dO"], None, out=outs)
    binding.tvm_attn_check_status()
    packed = {k: v.contiguous() for k, v in dev.items()}
    fwp = binding.tvm_attn_jvp_fwd(packed["Q"], packed["K"], packed["V"], packed["tQ"], packed["tK"], packed["tV"])
    ref = binding.tvm_attn_jvp_bwd(packed["Q"], packed["K"], packed["V"], packed["tQ"], packed["tK"], packed["tV"], *fwp,
                                   packed["dO"], None)
    for a, b in zip(outs, ref):
        assert torch.equal(a, b)
    assert not outs[3].any() and not outs[4].any() and not outs[5].any()


def test_strides_that_cannot_be_read_are_refused():
    lib = binding.load()
    import ctypes
    p = binding.Params(1, 2, 64, 32, 0.0, binding.BF16, 0, 0)
    p.q_strides[:] = (36, 8, 4096)        # row stride not a multiple of 8 elements
    assert lib.tvm_attn_jvp_workspace_bytes(ctypes.byref(p), 1) == 0
    p.q_strides[:] = (16, 32, 4096)       # row stride below d: rows would overlap
    assert lib.tvm_attn_jvp_workspace_bytes(ctypes.byref(p), 1) == 0
    p.q_strides[:] = (64, 32, 8192)
    assert lib.tvm_attn_jvp_workspace_bytes(ctypes.byref(p), 1) == 3 * 4 * 2 * 64
    big = binding.Params(1, 1, 64, 128, 0.0, binding.BF16, 0, 32)      # M != N at d = 128: not supported
    x = torch.zeros(1, 1, 32, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 1, 64, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.TvmAttnError) as e:
        binding.tvm_attn_jvp_fwd(x, k, k, x, k, k)
    assert e.value.code == -2 and big.M == 32
