"""Pins for the CPU oracle: nothing here touches the CUDA path.

Both writings of the oracle (whole-matrix numpy, row-at-a-time C) are checked against things
the mathematics fixes independently of them: finite differences, automatic differentiation of
the plain definition by a library, closed forms, invariants and library routines.
"""
import numpy as np
import pytest
import scipy.special
import torch

from oracle import attn_jvp_numpy as onp
from oracle import c_oracle as oc


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _inputs(B, H, N, d, seed=0, n=8):
    return [_rand((B, H, N, d), seed * 100 + k) for k in range(n)]


def _fwd_np(*a):
    return onp.attn_jvp_fwd(*a)


def _fwd_c(*a):
    return oc.attn_jvp_fwd(*a)[:4]


def _bwd_np(*a):
    return onp.attn_jvp_bwd(*a)


def _bwd_c(*a):
    return oc.attn_jvp_bwd(*a)[:6]


FWDS = [pytest.param(_fwd_np, id="numpy"), pytest.param(_fwd_c, id="c")]
BWDS = [pytest.param(_bwd_np, id="numpy"), pytest.param(_bwd_c, id="c")]
PAIRS = [pytest.param(_fwd_np, _bwd_np, id="numpy"), pytest.param(_fwd_c, _bwd_c, id="c")]


def _close(a, b, tol):
    scale = max(1.0, float(np.abs(b).max()))
    assert float(np.abs(a - b).max()) <= tol * scale, (float(np.abs(a - b).max()), tol * scale)


# ---------------------------------------------------------------- two writings agree

def test_c_and_numpy_writings_agree_on_tiny():
    xs = _inputs(2, 2, 64, 32)
    alpha = 1 / np.sqrt(32)
    for a, b in zip(_fwd_c(*xs[:6], alpha), _fwd_np(*xs[:6], alpha)):
        _close(a, b, 1e-12)
    for a, b in zip(_bwd_c(*xs, alpha), _bwd_np(*xs, alpha)):
        _close(a, b, 1e-12)


def test_c_oracle_thread_count_does_not_change_results():
    xs = _inputs(3, 2, 17, 8, seed=3)
    r1 = oc.attn_jvp_bwd(*xs, 0.3, nthreads=1)
    r4 = oc.attn_jvp_bwd(*xs, 0.3, nthreads=4)
    assert r1[6] == 1 and r4[6] == 4
    for a, b in zip(r1[:6], r4[:6]):
        assert np.array_equal(a, b)


# ---------------------------------------------------------------- forward pins

def test_rowsum_invariants_of_P_and_Pdot():
    Q, K, V, tQ, tK, tV = _inputs(1, 2, 33, 8, seed=1, n=6)
    _, P, _, _, _, Pd, _ = onp.scores(Q, K, tQ, tK, 0.4)
    _close(P.sum(-1), np.ones_like(P.sum(-1)), 1e-14)
    _close(Pd.sum(-1), np.zeros_like(Pd.sum(-1)), 1e-14)


@pytest.mark.parametrize("fwd", FWDS)
def test_rowsum_invariants_through_outputs(fwd):
    # V = all ones: O = rowsum(P) = 1; tV = 0: tO = rowsum(Pdot) = 0.
    Q, K, _, tQ, tK, _ = _inputs(1, 2, 33, 8, seed=2, n=6)
    V = np.ones_like(Q)
    O, tO, _, _ = fwd(Q, K, V, tQ, tK, np.zeros_like(Q), 0.4)
    _close(O, np.ones_like(O), 1e-14)
    _close(tO, np.zeros_like(tO), 1e-14)


@pytest.mark.parametrize("fwd", FWDS)
def test_tangents_zero_gives_textbook_softmax_attention(fwd):
    Q, K, V = _inputs(2, 1, 19, 8, seed=4, n=3)
    z = np.zeros_like(Q)
    alpha = 0.37
    O, tO, lse, mu = fwd(Q, K, V, z, z, z, alpha)
    A = alpha * np.einsum("bhid,bhjd->bhij", Q, K)
    _close(O, scipy.special.softmax(A, axis=-1) @ V, 1e-13)
    _close(lse, scipy.special.logsumexp(A, axis=-1), 1e-13)
    assert np.abs(tO).max() == 0.0 and np.abs(mu).max() == 0.0


@pytest.mark.parametrize("fwd", FWDS)
def test_tO_is_central_finite_difference_of_O(fwd):
    Q, K, V, tQ, tK, tV = _inputs(1, 2, 12, 6, seed=5, n=6)
    alpha, eps = 0.41, 1e-5
    z = np.zeros_like(Q)
    _, tO, lse, mu = fwd(Q, K, V, tQ, tK, tV, alpha)
    Op, _, lp, _ = fwd(Q + eps * tQ, K + eps * tK, V + eps * tV, z, z, z, alpha)
    Om, _, lm, _ = fwd(Q - eps * tQ, K - eps * tK, V - eps * tV, z, z, z, alpha)
    _close(tO, (Op - Om) / (2 * eps), 1e-8)
    # mu is the directional derivative of the log-sum-exp.
    _close(mu, (lp - lm) / (2 * eps), 1e-8)


@pytest.mark.parametrize("fwd", FWDS)
def test_tO_is_linear_in_the_tangents(fwd):
    Q, K, V, t1q, t1k, t1v, t2q, t2k = _inputs(1, 2, 10, 4, seed=6)
    t2v = _rand(Q.shape, 999)
    a, b, alpha = 0.7, -1.9, 0.5
    tO1 = fwd(Q, K, V, t1q, t1k, t1v, alpha)[1]
    tO2 = fwd(Q, K, V, t2q, t2k, t2v, alpha)[1]
    tO12 = fwd(Q, K, V, a * t1q + b * t2q, a * t1k + b * t2k, a * t1v + b * t2v, alpha)[1]
    _close(tO12, a * tO1 + b * tO2, 1e-13)


@pytest.mark.parametrize("fwd", FWDS)
def test_special_cases_of_the_forward(fwd):
    Q, K, V, tQ, tK, tV = _inputs(1, 2, 9, 4, seed=7, n=6)
    z = np.zeros_like(Q)
    alpha = 0.6
    # tQ = tK = 0: P has no tangent, tO = attention(Q, K, tV).
    O_tv = fwd(Q, K, tV, z, z, z, alpha)[0]
    _close(fwd(Q, K, V, z, z, tV, alpha)[1], O_tv, 1e-14)
    # V rows identical: Pdot V = rowsum(Pdot) v = 0, so tO = P tV.
    Vc = np.broadcast_to(V[:, :, :1, :], V.shape).copy()
    _close(fwd(Q, K, Vc, tQ, tK, tV, alpha)[1], O_tv, 1e-13)
    # alpha = 0: uniform P, no dependence on Q, K or their tangents.
    O0, tO0, lse0, mu0 = fwd(Q, K, V, tQ, tK, tV, 0.0)
    _close(O0, np.broadcast_to(V.mean(2, keepdims=True), V.shape), 1e-14)
    _close(tO0, np.broadcast_to(tV.mean(2, keepdims=True), V.shape), 1e-14)
    _close(lse0, np.full_like(lse0, np.log(9)), 1e-14)
    # N = 1: O = V, tO = tV.
    q1, k1, v1, a1, b1, c1 = [x[:, :, :1, :].copy() for x in (Q, K, V, tQ, tK, tV)]
    O1, tO1, _, _ = fwd(q1, k1, v1, a1, b1, c1, alpha)
    _close(O1, v1, 1e-15)
    _close(tO1, c1, 1e-15)


@pytest.mark.parametrize("fwd", FWDS)
def test_identical_keys_closed_form(fwd):
    # All keys equal: P = 1/N, and tO_i = (1/N) sum_j alpha <Q_i, tK_j - mean tK> V_j + mean tV
    # (the tQ term is constant over j and cancels against mu).
    Q, K, V, tQ, tK, tV = _inputs(1, 1, 7, 5, seed=8, n=6)
    K = np.broadcast_to(K[:, :, :1, :], K.shape).copy()
    alpha = 0.8
    O, tO, _, _ = fwd(Q, K, V, tQ, tK, tV, alpha)
    n = 7
    tKc = tK - tK.mean(2, keepdims=True)
    coef = alpha * np.einsum("bhid,bhjd->bhij", Q, tKc) / n
    _close(O, np.broadcast_to(V.mean(2, keepdims=True), V.shape), 1e-14)
    _close(tO, coef @ V + tV.mean(2, keepdims=True), 1e-13)


@pytest.mark.parametrize("fwd", FWDS)
def test_key_permutation_invariance(fwd):
    Q, K, V, tQ, tK, tV = _inputs(1, 1, 11, 4, seed=9, n=6)
    perm = np.random.default_rng(1).permutation(11)
    r0 = fwd(Q, K, V, tQ, tK, tV, 0.5)
    r1 = fwd(Q, K[:, :, perm], V[:, :, perm], tQ, tK[:, :, perm], tV[:, :, perm], 0.5)
    for a, b in zip(r0, r1):
        _close(a, b, 1e-13)


# ---------------------------------------------------------------- backward pins

def _loss(fwd, xs, G, Hc, alpha):
    O, tO, _, _ = fwd(*xs, alpha)
    return float((G * O).sum() + (Hc * tO).sum())


@pytest.mark.parametrize("fwd,bwd", PAIRS)
def test_every_gradient_element_against_finite_differences_micro(fwd, bwd):
    xs = _inputs(1, 1, 8, 4, seed=10, n=6)
    G, Hc = _rand(xs[0].shape, 77), _rand(xs[0].shape, 78)
    alpha, eps = 0.5, 1e-5
    grads = bwd(*xs, G, Hc, alpha)
    order = [0, 1, 2, 3, 4, 5]  # dQ, dK, dV, dtQ, dtK, dtV  <->  inputs Q, K, V, tQ, tK, tV
    for gi, xi in zip(range(6), order):
        fd = np.zeros_like(xs[xi])
        it = np.nditer(xs[xi], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = xs[xi][idx]
            xs[xi][idx] = keep + eps
            lp = _loss(fwd, xs, G, Hc, alpha)
            xs[xi][idx] = keep - eps
            lm = _loss(fwd, xs, G, Hc, alpha)
            xs[xi][idx] = keep
            fd[idx] = (lp - lm) / (2 * eps)
        _close(grads[gi], fd, 2e-8)


@pytest.mark.parametrize("fwd,bwd", PAIRS)
def test_gradients_against_directional_finite_differences_tiny(fwd, bwd):
    xs = _inputs(2, 2, 64, 32, seed=0, n=6)
    G, Hc = _rand(xs[0].shape, 11), _rand(xs[0].shape, 12)
    alpha, eps = 1 / np.sqrt(32), 1e-5
    grads = bwd(*xs, G, Hc, alpha)
    for gi in range(6):
        for k in range(8):
            u = _rand(xs[gi].shape, 500 + 10 * gi + k)
            keep = xs[gi]
            xs[gi] = keep + eps * u
            lp = _loss(fwd, xs, G, Hc, alpha)
            xs[gi] = keep - eps * u
            lm = _loss(fwd, xs, G, Hc, alpha)
            xs[gi] = keep
            fd = (lp - lm) / (2 * eps)
            an = float((grads[gi] * u).sum())
            assert abs(fd - an) <= 1e-7 * max(1.0, abs(an)), (gi, k, fd, an)


def _torch_vanilla(xs, G, Hc, alpha):
    """Explicit-math SDPA under torch.func.jvp + autograd in fp64 (the paper's 'vanilla' path)."""
    t = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in xs]

    def sdpa(q, k, v):
        return torch.softmax(alpha * q @ k.transpose(-1, -2), dim=-1) @ v

    O, tO = torch.func.jvp(sdpa, (t[0], t[1], t[2]), (t[3], t[4], t[5]))
    loss = (torch.tensor(G) * O).sum() + (torch.tensor(Hc) * tO).sum()
    grads = torch.autograd.grad(loss, t)
    return O.detach().numpy(), tO.detach().numpy(), [g.numpy() for g in grads]


@pytest.mark.parametrize("fwd,bwd", PAIRS)
def test_against_torch_jvp_and_autograd_of_the_plain_definition(fwd, bwd):
    for (B, H, N, d, seed) in [(1, 1, 7, 5, 20), (2, 2, 64, 32, 21), (1, 3, 37, 24, 22)]:
        xs = _inputs(B, H, N, d, seed=seed, n=6)
        G, Hc = _rand(xs[0].shape, seed + 50), _rand(xs[0].shape, seed + 51)
        alpha = 1 / np.sqrt(d)
        O_t, tO_t, g_t = _torch_vanilla(xs, G, Hc, alpha)
        O, tO, _, _ = fwd(*xs, alpha)
        _close(O, O_t, 1e-13)
        _close(tO, tO_t, 1e-12)
        for a, b in zip(bwd(*xs, G, Hc, alpha), g_t):
            _close(a, b, 1e-12)


@pytest.mark.parametrize("bwd", BWDS)
def test_zero_tangent_cotangent_gives_textbook_attention_backward(bwd):
    xs = _inputs(1, 2, 13, 8, seed=30, n=6)
    G = _rand(xs[0].shape, 31)
    alpha = 0.35
    q, k, v = [torch.tensor(x, requires_grad=True) for x in xs[:3]]
    out = torch.nn.functional.scaled_dot_product_attention(q, k, v, scale=alpha)
    gq, gk, gv = torch.autograd.grad((out * torch.tensor(G)).sum(), (q, k, v))
    dQ, dK, dV, dtQ, dtK, dtV = bwd(*xs, G, np.zeros_like(G), alpha)
    _close(dQ, gq.numpy(), 1e-12)
    _close(dK, gk.numpy(), 1e-12)
    _close(dV, gv.numpy(), 1e-12)
    assert max(np.abs(x).max() for x in (dtQ, dtK, dtV)) == 0.0


@pytest.mark.parametrize("bwd", BWDS)
def test_single_key_backward(bwd):
    xs = _inputs(2, 1, 1, 6, seed=32, n=6)
    G, Hc = _rand(xs[0].shape, 33), _rand(xs[0].shape, 34)
    dQ, dK, dV, dtQ, dtK, dtV = bwd(*xs, G, Hc, 0.7)
    _close(dV, G, 1e-15)
    _close(dtV, Hc, 1e-15)
    for x in (dQ, dK, dtQ, dtK):
        _close(x, np.zeros_like(x), 1e-14)


def test_row_sum_shortcuts_hold():
    # Sigma_1 = rowsum(Hc*O), Sigma_2 = rowsum(Hc*tO), d0 = rowsum(G*O): what a kernel may use
    # instead of the N x N sweeps of App. C Step 1.
    Q, K, V, tQ, tK, tV, G, Hc = _inputs(1, 2, 21, 8, seed=35)
    alpha = 0.45
    _, P, _, _, Nn, _, _ = onp.scores(Q, K, tQ, tK, alpha)
    O, tO, _, _ = onp.attn_jvp_fwd(Q, K, V, tQ, tK, tV, alpha)
    D = Hc @ np.swapaxes(V, -1, -2)
    HtV = Hc @ np.swapaxes(tV, -1, -2)
    _close((P * D).sum(-1), (Hc * O).sum(-1), 1e-13)
    _close((P * (HtV + D * Nn)).sum(-1), (Hc * tO).sum(-1), 1e-13)
    _close((P * (G @ np.swapaxes(V, -1, -2))).sum(-1), (G * O).sum(-1), 1e-13)


@pytest.mark.parametrize("bwd", BWDS)
def test_tangent_path_matches_the_six_step_equations(bwd):
    """With dO = 0 the gradients are App. C steps 2-6 as printed (index slips in steps 4 and 6
    read as sum over i and Q_{i,:}); mu/l there is the normalised mu."""
    Q, K, V, tQ, tK, tV, _, Hc = _inputs(1, 1, 10, 4, seed=36)
    alpha = 0.55
    _, P, T, mu, _, _, _ = onp.scores(Q, K, tQ, tK, alpha)
    P, T, mu = P[0, 0], T[0, 0], mu[0, 0]
    q, k, v, tq, tk, tv, h = [x[0, 0] for x in (Q, K, V, tQ, tK, tV, Hc)]
    n = 10
    HV, HtV = h @ v.T, h @ tv.T
    Nn = T - mu[:, None]
    s1 = np.array([sum(P[i, j] * HV[i, j] for j in range(n)) for i in range(n)])
    s2 = np.array([sum(P[i, j] * (HtV[i, j] + HV[i, j] * Nn[i, j]) for j in range(n)) for i in range(n)])
    br23 = (HV - s1[:, None]) * P
    br45 = ((-s1[:, None]) * T + s1[:, None] * mu[:, None]) * P \
        + (HtV + HV * (T - mu[:, None]) - s2[:, None]) * P
    dK1 = alpha * br23.T @ tq
    dtK = alpha * br23.T @ q
    dQ1 = alpha * br23 @ tk
    dtQ = alpha * br23 @ k
    dK = dK1 + alpha * br45.T @ q
    dQ = dQ1 + alpha * br45 @ k
    dtV = P.T @ h
    dV = (P * Nn).T @ h
    got = bwd(Q, K, V, tQ, tK, tV, np.zeros_like(Hc), Hc, alpha)
    for a, b in zip(got, (dQ, dK, dV, dtQ, dtK, dtV)):
        _close(a[0, 0], b, 1e-13)


def test_numpy_oracle_accepts_a_subset_of_query_rows():
    """Queries are independent of one another (App. C Eq. "sdpa": one softmax per query row), so the numpy
    oracle called with fewer query rows than keys must return exactly those rows of O, tO, lse, mu, dQ, dtQ.
    The GPU test of the longest sequence relies on this."""
    xs = _inputs(1, 2, 23, 8, seed=11)
    rows = [0, 7, 22]
    sub = lambda a: np.ascontiguousarray(a[:, :, rows])
    Q, K, V, tQ, tK, tV, G, Hc = xs
    full_f = onp.attn_jvp_fwd(Q, K, V, tQ, tK, tV, 0.37)
    part_f = onp.attn_jvp_fwd(sub(Q), K, V, sub(tQ), tK, tV, 0.37)
    for a, b in zip(part_f, full_f):
        _close(a, b[:, :, rows], 1e-14)
    full_b = onp.attn_jvp_bwd(Q, K, V, tQ, tK, tV, G, Hc, 0.37)
    part_b = onp.attn_jvp_bwd(sub(Q), K, V, sub(tQ), tK, tV, sub(G), sub(Hc), 0.37)
    _close(part_b[0], full_b[0][:, :, rows], 1e-14)
    _close(part_b[3], full_b[3][:, :, rows], 1e-14)


@pytest.mark.parametrize("bwd", BWDS)
def test_query_rows_with_zero_cotangents_contribute_nothing(bwd):
    """A query row whose cotangents dO and dtO are zero adds nothing to any key-side gradient (every term of
    App. C steps 2, 4 and 6 carries a factor from that row of the cotangents) and gets zero dQ, dtQ.  So the
    key-side gradients of a problem whose cotangents live on a few rows are those of the few-row problem:
    the GPU test at S = 32,768 relies on this to check every element of dK, dtK, dV, dtV."""
    xs = _inputs(1, 2, 29, 8, seed=13)
    rows = [2, 11, 28]
    mask = np.zeros((1, 1, 29, 1))
    mask[:, :, rows] = 1.0
    Q, K, V, tQ, tK, tV, G, Hc = xs
    G, Hc = G * mask, Hc * mask
    full = bwd(Q, K, V, tQ, tK, tV, G, Hc, 0.41)
    sub = lambda a: np.ascontiguousarray(a[:, :, rows])
    part = onp.attn_jvp_bwd(sub(Q), K, V, sub(tQ), tK, tV, sub(G), sub(Hc), 0.41)
    for i in (1, 2, 4, 5):                      # dK, dV, dtK, dtV
        _close(part[i], full[i], 1e-13)
    others = [i for i in range(29) if i not in rows]
    for i in (0, 3):                            # dQ, dtQ
        _close(part[i], full[i][:, :, rows], 1e-13)
        assert not np.any(full[i][:, :, others])
