"""fp64 numpy oracle for attention with a Jacobian-vector product and its backward pass.

TEST INFRASTRUCTURE ONLY.  This module is the slow, whole-matrix CPU definition that the
CUDA path is compared against.  It shares no code with the CUDA path and must never be
imported by the product package; only tests, the smoke check and the CPU-baseline leg of
the benchmark may call it.

What it computes, per (batch, head), everything in float64 (paper App. C, Eq. "sdpa" and the
definitions of P, S, N, S-dot and mu under "Step 1"):

    A   = alpha * Q K^T                      scaled scores
    P   = softmax_rows(A)                    exact two-pass softmax, N x N materialised
    O   = P V                                primal output (operand order of Eq. "sdpa" read as P V)
    T   = alpha * (tQ K^T + Q tK^T)          tangent of the scaled scores (alpha * S-dot)
    mu  = rowsum(P * T)                      P-weighted mean of T per query row
    Nn  = T - mu                             the paper's N_ij (mu here already normalised)
    Pd  = P * Nn                             tangent of P
    tO  = Pd V + P tV                        tangent output = directional derivative of O
    lse = log rowsum(exp(A))                 natural-log normaliser of the scaled scores

Backward of a scalar loss L(O, tO) with G = dL/dO and Hc = dL/d(tO) (paper App. C steps 1-6 for
the tangent path; the primal path of a standard attention backward is added in, as the paper
says the two are summed):

    D   = Hc V^T                X = G V^T + Hc tV^T
    Sg1 = rowsum(P * D)                                   (Step 1, Sigma_1)
    Sg2 = rowsum(P * (Hc tV^T + D * Nn))                  (Step 1, Sigma_2)
    d0  = rowsum(P * (G V^T))                             (standard attention backward row term)
    W   = P * (D - Sg1)                                   = dL/dT
    dA  = P * (X - d0 - Sg2) + W * Nn                     = dL/dA (second-order terms via Pd)
    dV  = P^T G + Pd^T Hc       dtV = P^T Hc              (Step 6 + primal part)
    dQ  = alpha (dA K + W tK)   dtQ = alpha W K           (Steps 3, 5 + primal part)
    dK  = alpha (dA^T Q + W^T tQ)   dtK = alpha W^T Q     (Steps 2, 4 + primal part)
"""
import numpy as np


def _check(*xs):
    for x in xs:
        if x.dtype != np.float64 or x.ndim != 4:
            raise ValueError("oracle expects float64 arrays of shape (B, H, N, d)")


def scores(Q, K, tQ, tK, alpha):
    """A, P, T, mu, Nn, Pd as full (B,H,N,N) matrices (definitions under App. C 'Step 1')."""
    A = alpha * np.einsum("bhid,bhjd->bhij", Q, K)
    m = A.max(axis=-1, keepdims=True)
    E = np.exp(A - m)
    rowsum = E.sum(axis=-1, keepdims=True)
    P = E / rowsum
    lse = (m + np.log(rowsum))[..., 0]
    T = alpha * (np.einsum("bhid,bhjd->bhij", tQ, K) + np.einsum("bhid,bhjd->bhij", Q, tK))
    mu = (P * T).sum(axis=-1)
    Nn = T - mu[..., None]
    Pd = P * Nn
    return A, P, T, mu, Nn, Pd, lse


def attn_jvp_fwd(Q, K, V, tQ, tK, tV, alpha):
    """Returns O, tO (B,H,N,d) and lse, mu (B,H,N)."""
    _check(Q, K, V, tQ, tK, tV)
    _, P, _, mu, _, Pd, lse = scores(Q, K, tQ, tK, alpha)
    O = P @ V
    tO = Pd @ V + P @ tV
    return O, tO, lse, mu


def attn_jvp_bwd(Q, K, V, tQ, tK, tV, G, Hc, alpha):
    """Returns dQ, dK, dV, dtQ, dtK, dtV for cotangents G = dL/dO, Hc = dL/d(tO)."""
    _check(Q, K, V, tQ, tK, tV, G, Hc)
    _, P, _, _, Nn, Pd, _ = scores(Q, K, tQ, tK, alpha)
    Vt = np.swapaxes(V, -1, -2)
    tVt = np.swapaxes(tV, -1, -2)
    D = Hc @ Vt
    GV = G @ Vt
    HtV = Hc @ tVt
    Sg1 = (P * D).sum(axis=-1, keepdims=True)
    Sg2 = (P * (HtV + D * Nn)).sum(axis=-1, keepdims=True)
    d0 = (P * GV).sum(axis=-1, keepdims=True)
    W = P * (D - Sg1)
    dA = P * (GV + HtV - d0 - Sg2) + W * Nn
    Pt = np.swapaxes(P, -1, -2)
    dV = Pt @ G + np.swapaxes(Pd, -1, -2) @ Hc
    dtV = Pt @ Hc
    dQ = alpha * (dA @ K + W @ tK)
    dtQ = alpha * (W @ K)
    dAt = np.swapaxes(dA, -1, -2)
    Wt = np.swapaxes(W, -1, -2)
    dK = alpha * (dAt @ Q + Wt @ tQ)
    dtK = alpha * (Wt @ Q)
    return dQ, dK, dV, dtQ, dtK, dtV
