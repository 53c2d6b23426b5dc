"""fp64 numpy oracle for RMSNorm QK-normalisation with a tangent (JVP) and its backward pass.

TEST INFRASTRUCTURE ONLY.  Slow, plain definitions that the CUDA kernels of the attention prologue are
compared against.  Shares no code with the CUDA path and must never be imported by the product package.

What it computes, per row x in R^d of a (B, H, N, d) tensor, everything in float64 (paper Sec. 4,
"semi-Lipschitz control": RMSNorm as QK-norm with a learnable scale; App. "Lipschitzness of RMSNorm"
for the definition and the Jacobian):

    r  = sqrt(mean(x^2) + eps)              RMS(x); the paper prints the sum without the square, its own
                                            Jacobian is that of the squared form, which is what is used here
    u  = x / r                              RMSNorm(x)
    y  = g * u                              QK-norm: learnable per-channel scale g in R^d, shared by all rows
    J  = (I - u u^T / d) / r                Jacobian of u with respect to x (the paper's last displayed form)
    ty = g * (J tx)                         tangent of y along the input tangent tx (g carries no tangent:
                                            the tangent direction of the method is the time argument)

Backward of a scalar loss L(y, ty) with cotangents dy = dL/dy and dty = dL/d(ty):

    dtx = J (g * dty)                       J is symmetric
    dx  = J (g * dy) + d/dx [ (g * dty) . (J(x) tx) ]        the second term differentiates J itself
    dg  = sum over rows of  dy * u + dty * (J tx)
"""
import numpy as np


def _rms(x, eps):
    return np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)


def rmsnorm_jvp_fwd(x, tx, g, eps):
    """y, ty for x, tx of shape (..., d) and g of shape (d,)."""
    d = x.shape[-1]
    r = _rms(x, eps)
    u = x / r
    Jtx = tx / r - u * (u * tx).sum(axis=-1, keepdims=True) / (d * r)
    return g * u, g * Jtx


def rmsnorm_jvp_bwd(x, tx, g, dy, dty, eps):
    """dx, dtx (shape of x) and dg (shape (d,))."""
    d = x.shape[-1]
    r = _rms(x, eps)
    u = x / r
    a = g * dy
    b = g * dty

    def J(v):
        return v / r - u * (u * v).sum(axis=-1, keepdims=True) / (d * r)

    dtx = J(b)
    # derivative of f(x) = tx / r - x (x . tx) / (d r^3) contracted with b, term by term:
    #   d(1/r)/dx = -x / (d r^3),  d(r^-3)/dx = -3 x / (d r^5)
    s = (x * tx).sum(axis=-1, keepdims=True)
    bx = (b * x).sum(axis=-1, keepdims=True)
    bt = (b * tx).sum(axis=-1, keepdims=True)
    dx_t = (-bt * x / (d * r ** 3)                 # from tx / r
            - b * s / (d * r ** 3)                 # from the leading x of  x (x . tx)
            - bx * tx / (d * r ** 3)               # from (x . tx)
            + 3.0 * bx * s * x / (d * d * r ** 5)) # from r^-3
    dx = J(a) + dx_t
    Jtx = J(tx)
    dg = (dy * u + dty * Jtx).reshape(-1, d).sum(axis=0)
    return dx, dtx, dg
