"""Pins of the RMSNorm QK-normalisation oracle (oracle/qk_rmsnorm_numpy.py) to things other than itself:
library routines, finite differences, torch autograd through torch.func.jvp of the plain definition, closed
forms and invariants.  A dropped term, a wrong sign or a wrong power of r in the oracle fails several of them.
"""
import numpy as np
import torch

from oracle import qk_rmsnorm_numpy as orn


def _data(shape=(2, 3, 5, 8), seed=0):
    rng = np.random.default_rng(seed)
    x, tx, dy, dty = (rng.standard_normal(shape) for _ in range(4))
    g = rng.standard_normal(shape[-1]) + 1.5
    return x, tx, g, dy, dty


def test_primal_is_torch_rms_norm():
    x, tx, g, _, _ = _data()
    y, _ = orn.rmsnorm_jvp_fwd(x, tx, g, 1e-6)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (x.shape[-1],), torch.from_numpy(g), eps=1e-6).numpy()
    assert np.abs(y - ref).max() < 1e-13


def test_jacobian_is_the_one_the_paper_prints():
    """App. 'Lipschitzness of RMSNorm': d u_i / d x_j = delta_ij / r - x_i x_j / (d r^3), written out per element."""
    rng = np.random.default_rng(1)
    d = 6
    x = rng.standard_normal(d)
    eps = 0.01
    r = np.sqrt((x * x).mean() + eps)
    Jac = np.eye(d) / r - np.outer(x, x) / (d * r ** 3)
    for j in range(d):
        e = np.zeros(d)
        e[j] = 1.0
        _, col = orn.rmsnorm_jvp_fwd(x[None], e[None], np.ones(d), eps)
        assert np.abs(col[0] - Jac[:, j]).max() < 1e-14


def test_tangent_is_central_finite_difference():
    x, tx, g, _, _ = _data(seed=2)
    h = 1e-6
    yp, _ = orn.rmsnorm_jvp_fwd(x + h * tx, tx, g, 1e-5)
    ym, _ = orn.rmsnorm_jvp_fwd(x - h * tx, tx, g, 1e-5)
    _, ty = orn.rmsnorm_jvp_fwd(x, tx, g, 1e-5)
    assert np.abs((yp - ym) / (2 * h) - ty).max() < 1e-8


def test_invariants_without_epsilon():
    x, tx, g, _, _ = _data(seed=3)
    one = np.ones_like(g)
    u, tu = orn.rmsnorm_jvp_fwd(x, tx, one, 0.0)
    assert np.abs((u * u).mean(axis=-1) - 1.0).max() < 1e-14          # unit RMS
    assert np.abs((u * tu).sum(axis=-1)).max() < 1e-13                 # the tangent stays on the sphere
    u2, tu2 = orn.rmsnorm_jvp_fwd(3.7 * x, 3.7 * tx, one, 0.0)           # scale invariance of the input
    assert np.abs(u2 - u).max() < 1e-14 and np.abs(tu2 - tu).max() < 1e-13
    _, tpar = orn.rmsnorm_jvp_fwd(x, 2.5 * x, one, 0.0)                  # moving along x changes nothing
    assert np.abs(tpar).max() < 1e-13
    a, b = 0.3, -1.2                                                     # linear in the tangent
    tx2 = np.random.default_rng(9).standard_normal(x.shape)
    _, t12 = orn.rmsnorm_jvp_fwd(x, a * tx + b * tx2, g, 1e-3)
    _, t1 = orn.rmsnorm_jvp_fwd(x, tx, g, 1e-3)
    _, t2 = orn.rmsnorm_jvp_fwd(x, tx2, g, 1e-3)
    assert np.abs(t12 - (a * t1 + b * t2)).max() < 1e-13


def test_large_epsilon_limit_is_a_plain_scaling():
    """With eps far above mean(x^2), r -> sqrt(eps): y = g x / sqrt(eps) and ty = g tx / sqrt(eps)."""
    x, tx, g, _, _ = _data(seed=4)
    eps = 1e12
    y, ty = orn.rmsnorm_jvp_fwd(x, tx, g, eps)
    assert np.abs(y * np.sqrt(eps) - g * x).max() < 1e-9
    assert np.abs(ty * np.sqrt(eps) - g * tx).max() < 1e-9


def test_every_gradient_element_against_finite_differences():
    x, tx, g, dy, dty = _data(shape=(1, 2, 3, 4), seed=5)
    eps = 1e-3

    def loss(x_, tx_, g_):
        y, ty = orn.rmsnorm_jvp_fwd(x_, tx_, g_, eps)
        return float((dy * y).sum() + (dty * ty).sum())

    dx, dtx, dg = orn.rmsnorm_jvp_bwd(x, tx, g, dy, dty, eps)
    h = 1e-6
    for arr, grad, which in ((x, dx, 0), (tx, dtx, 1), (g, dg, 2)):
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            args = [x.copy(), tx.copy(), g.copy()]
            args[which][idx] += h
            up = loss(*args)
            args[which][idx] -= 2 * h
            dn = loss(*args)
            assert abs((up - dn) / (2 * h) - grad[idx]) < 2e-7, (which, idx)


def test_against_torch_jvp_and_autograd_of_the_plain_definition():
    x, tx, g, dy, dty = _data(seed=6)
    eps = 1e-4
    xt, txt, gt = (torch.from_numpy(a).requires_grad_(True) for a in (x, tx, g))

    def f(x_):
        return gt * x_ / torch.sqrt((x_ * x_).mean(dim=-1, keepdim=True) + eps)

    y, ty = torch.func.jvp(f, (xt,), (txt,))
    L = (torch.from_numpy(dy) * y).sum() + (torch.from_numpy(dty) * ty).sum()
    rx, rtx, rg = torch.autograd.grad(L, (xt, txt, gt))
    oy, oty = orn.rmsnorm_jvp_fwd(x, tx, g, eps)
    dx, dtx, dg = orn.rmsnorm_jvp_bwd(x, tx, g, dy, dty, eps)
    assert np.abs(oy - y.detach().numpy()).max() < 1e-13 and np.abs(oty - ty.detach().numpy()).max() < 1e-13
    assert np.abs(dx - rx.numpy()).max() < 1e-12
    assert np.abs(dtx - rtx.numpy()).max() < 1e-12
    assert np.abs(dg - rg.numpy()).max() < 1e-12


def test_zero_tangent_cotangent_gives_the_textbook_rmsnorm_backward():
    """dty = 0: dx = (a - u (a . u) / d) / r with a = g dy, dtx = 0, dg = sum dy u."""
    x, tx, g, dy, _ = _data(seed=7)
    eps = 1e-5
    d = x.shape[-1]
    dx, dtx, dg = orn.rmsnorm_jvp_bwd(x, tx, g, dy, np.zeros_like(dy), eps)
    r = np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    u = x / r
    a = g * dy
    assert np.abs(dx - (a - u * (a * u).sum(-1, keepdims=True) / d) / r).max() < 1e-14
    assert not dtx.any()
    assert np.abs(dg - (dy * u).reshape(-1, d).sum(0)).max() < 1e-13
