"""Builds (gcc) and wraps the plain-C fp64 oracle in attn_jvp_oracle.c.

TEST INFRASTRUCTURE ONLY: used by tests, the smoke check and the CPU-baseline leg of the
benchmark.  Arguments and results are numpy float64 arrays shaped (B, H, N, d) / (B, H, N).
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_jvp_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_OUT = os.path.join(_OUT_DIR, "liboracle_attn_jvp.so")
_lib = None


def build(force=False):
    """Compile the C oracle with gcc -O2 (no fast-math); returns the path of the shared object."""
    if not force and os.path.exists(_OUT) and os.path.getmtime(_OUT) >= os.path.getmtime(_SRC):
        return _OUT
    os.makedirs(_OUT_DIR, exist_ok=True)
    tmp = _OUT + ".tmp.%d" % os.getpid()
    subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread", _SRC, "-lm", "-o", tmp],
                   check=True)
    os.replace(tmp, _OUT)
    return _OUT


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.oracle_attn_jvp_fwd.restype = ctypes.c_int
        lib.oracle_attn_jvp_fwd.argtypes = [ctypes.c_long] * 3 + [ctypes.c_double] + [dp] * 10 + [ctypes.c_int]
        lib.oracle_attn_jvp_bwd.restype = ctypes.c_int
        lib.oracle_attn_jvp_bwd.argtypes = [ctypes.c_long] * 3 + [ctypes.c_double] + [dp] * 14 + [ctypes.c_int]
        _lib = lib
    return _lib


def _p(x):
    return x.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _prep(xs):
    out = [np.ascontiguousarray(x, dtype=np.float64) for x in xs]
    shape = out[0].shape
    if len(shape) != 4 or any(x.shape != shape for x in out):
        raise ValueError("oracle expects equal-shaped (B, H, N, d) arrays")
    return out, shape


def default_threads():
    return os.cpu_count() or 1


def attn_jvp_fwd(Q, K, V, tQ, tK, tV, alpha, nthreads=None):
    """Returns (O, tO, lse, mu, threads_used)."""
    (Q, K, V, tQ, tK, tV), (B, H, N, d) = _prep([Q, K, V, tQ, tK, tV])
    O = np.empty((B, H, N, d)); tO = np.empty((B, H, N, d))
    lse = np.empty((B, H, N)); mu = np.empty((B, H, N))
    rc = _load().oracle_attn_jvp_fwd(B * H, N, d, float(alpha), _p(Q), _p(K), _p(V), _p(tQ), _p(tK),
                                     _p(tV), _p(O), _p(tO), _p(lse), _p(mu),
                                     int(nthreads or default_threads()))
    if rc <= 0:
        raise RuntimeError("oracle_attn_jvp_fwd failed with code %d" % rc)
    return O, tO, lse, mu, rc


def attn_jvp_bwd(Q, K, V, tQ, tK, tV, G, Hc, alpha, nthreads=None):
    """Returns (dQ, dK, dV, dtQ, dtK, dtV, threads_used)."""
    (Q, K, V, tQ, tK, tV, G, Hc), (B, H, N, d) = _prep([Q, K, V, tQ, tK, tV, G, Hc])
    outs = [np.empty((B, H, N, d)) for _ in range(6)]
    rc = _load().oracle_attn_jvp_bwd(B * H, N, d, float(alpha), _p(Q), _p(K), _p(V), _p(tQ), _p(tK),
                                     _p(tV), _p(G), _p(Hc), *[_p(o) for o in outs],
                                     int(nthreads or default_threads()))
    if rc <= 0:
        raise RuntimeError("oracle_attn_jvp_bwd failed with code %d" % rc)
    return (*outs, rc)
