"""ctypes binding of the C-ABI library declared in include/tvm_attn.h.

Argument marshalling only: every step of the path runs in the CUDA kernels of the library.
PyTorch provides device memory and streams.  There is no CPU or library fallback: if the
shared object is missing or a call fails, an exception is raised.
"""
import ctypes
import os

import torch

from . import build as _build

BF16 = 0
FP32 = 1
FLAG_CUDA_CORES = 1

_STATUS_NAMES = {0: "OK", -1: "INVALID_ARG", -2: "UNSUPPORTED", -3: "WORKSPACE_TOO_SMALL", -4: "CUDA_ERROR",
                 -5: "DEVICE_TIMEOUT", -6: "TOO_LARGE"}
NOALLOC_MAX_ROWS = 262144


class TvmAttnError(RuntimeError):
    def __init__(self, where, code, text):
        super().__init__("%s failed: %s (%d): %s" % (where, _STATUS_NAMES.get(code, "?"), code, text))
        self.code = code


class Params(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("d", ctypes.c_int32),
                ("scale", ctypes.c_float), ("dtype", ctypes.c_int32), ("flags", ctypes.c_uint32), ("M", ctypes.c_int32),
                ("q_strides", ctypes.c_int64 * 3), ("k_strides", ctypes.c_int64 * 3)]


_lib = None
EXPORTS = ("tvm_attn_jvp_workspace_bytes", "tvm_attn_jvp_fwd", "tvm_attn_jvp_bwd", "tvm_attn_jvp_bwd_noalloc",
           "tvm_attn_check_status", "tvm_attn_selftest_timeout",
           "tvm_qk_rmsnorm_jvp_fwd", "tvm_qk_rmsnorm_jvp_bwd", "tvm_qk_rmsnorm_jvp_workspace_bytes",
           "tvm_attn_launch_count", "tvm_attn_strerror", "tvm_attn_version", "tvm_attn_set_profiling",
           "tvm_attn_get_profile")


def library_path():
    """Path of the shared object; the environment variable TVM_ATTN_LIBRARY selects another build."""
    return os.environ.get("TVM_ATTN_LIBRARY") or _build.LIB_PATH


def load(build_if_missing=False):
    """Loads libtvm_attn.so (built in-tree by build.py).  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        if not build_if_missing:
            raise FileNotFoundError("%s is missing: run paper_2511_19797_b200/build.py (nvcc, sm_100a) first" % path)
        _build.build()
    lib = ctypes.CDLL(path)
    vp, pp = ctypes.c_void_p, ctypes.POINTER(Params)
    lib.tvm_attn_jvp_workspace_bytes.restype = ctypes.c_size_t
    lib.tvm_attn_jvp_workspace_bytes.argtypes = [pp, ctypes.c_int]
    lib.tvm_attn_jvp_fwd.restype = ctypes.c_int
    lib.tvm_attn_jvp_fwd.argtypes = [pp] + [vp] * 10 + [vp, ctypes.c_size_t, vp]
    lib.tvm_attn_jvp_bwd.restype = ctypes.c_int
    lib.tvm_attn_jvp_bwd.argtypes = [pp] + [vp] * 18 + [vp, ctypes.c_size_t, vp]
    lib.tvm_attn_jvp_bwd_noalloc.restype = ctypes.c_int
    lib.tvm_attn_jvp_bwd_noalloc.argtypes = [pp] + [vp] * 18 + [vp]
    lib.tvm_attn_check_status.restype = ctypes.c_int
    lib.tvm_attn_check_status.argtypes = [vp]
    lib.tvm_qk_rmsnorm_jvp_workspace_bytes.restype = ctypes.c_size_t
    lib.tvm_qk_rmsnorm_jvp_workspace_bytes.argtypes = [pp]
    lib.tvm_qk_rmsnorm_jvp_fwd.restype = ctypes.c_int
    lib.tvm_qk_rmsnorm_jvp_fwd.argtypes = [pp, ctypes.c_float] + [vp] * 10 + [vp]
    lib.tvm_qk_rmsnorm_jvp_bwd.restype = ctypes.c_int
    lib.tvm_qk_rmsnorm_jvp_bwd.argtypes = [pp, ctypes.c_float] + [vp] * 16 + [vp, ctypes.c_size_t, vp]
    lib.tvm_attn_selftest_timeout.restype = ctypes.c_int
    lib.tvm_attn_selftest_timeout.argtypes = [ctypes.c_uint64, vp]
    lib.tvm_attn_launch_count.restype = ctypes.c_uint64
    lib.tvm_attn_launch_count.argtypes = []
    lib.tvm_attn_strerror.restype = ctypes.c_char_p
    lib.tvm_attn_strerror.argtypes = [ctypes.c_int]
    lib.tvm_attn_version.restype = ctypes.c_int
    lib.tvm_attn_version.argtypes = []
    lib.tvm_attn_set_profiling.restype = ctypes.c_int
    lib.tvm_attn_set_profiling.argtypes = [ctypes.c_int]
    lib.tvm_attn_get_profile.restype = ctypes.c_int
    lib.tvm_attn_get_profile.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int]
    _lib = lib
    return lib


def _raise(where, code):
    raise TvmAttnError(where, code, load().tvm_attn_strerror(code).decode())


def _strides(t):
    """{row, head, batch} element strides of a (B, H, rows, d) tensor; zeros for the packed layout."""
    if t.stride(3) != 1 and t.shape[3] != 1:
        raise ValueError("the d elements of a row must be contiguous")
    if t.is_contiguous():
        return (0, 0, 0)
    return (t.stride(2), t.stride(1), t.stride(0))


def _params(q, scale, flags, k=None):
    """Parameters from a query-side tensor q (B, H, M, d) and, for M != N or strided layouts, a key-side tensor k."""
    if q.dim() != 4:
        raise ValueError("expected (B, H, rows, d) tensors")
    if q.dtype == torch.bfloat16:
        dt = BF16
    elif q.dtype == torch.float32:
        dt = FP32
    else:
        raise ValueError("tensors must be bfloat16 or float32")
    B, H, M, d = q.shape
    k = q if k is None else k
    if k.dim() != 4 or k.shape[0] != B or k.shape[1] != H or k.shape[3] != d:
        raise ValueError("query-side and key-side tensors must agree in B, H and d")
    N = k.shape[2]
    p = Params(B, H, N, d, float(scale), dt, int(flags), 0 if M == N else M)
    p.q_strides[:] = _strides(q)
    p.k_strides[:] = _strides(k)
    return p


def _check_tensors(ref, tensors):
    """Every tensor of one side shares shape, strides, dtype and device with the side's first tensor."""
    for t in tensors:
        if t.shape != ref.shape or t.dtype != ref.dtype or t.device != ref.device or t.stride() != ref.stride():
            raise ValueError("all tensors of one side must share shape, strides, dtype and device")
        if not t.is_cuda:
            raise ValueError("tensors must be CUDA tensors")
    if not ref.is_cuda:
        raise ValueError("tensors must be CUDA tensors")


def _like(t):
    """A new tensor with the shape AND the strides of t (torch.empty_like does not keep the strides of a slice)."""
    return torch.empty_strided(t.shape, t.stride(), dtype=t.dtype, device=t.device)


def _ptr(t):
    """Device address of a tensor, or a null pointer for None (an absent cotangent or an unwanted output)."""
    return None if t is None else t.data_ptr()


def _stream_ptr(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def tvm_attn_jvp_workspace_bytes(B, H, N, d, dtype=BF16, is_bwd=True, scale=0.0, flags=0):
    p = Params(B, H, N, d, float(scale), dtype, flags)
    return int(load().tvm_attn_jvp_workspace_bytes(ctypes.byref(p), 1 if is_bwd else 0))


def tvm_attn_jvp_fwd(Q, K, V, tQ, tK, tV, scale=0.0, flags=0, out=None, stream=None):
    """Forward: returns (O, tO, lse, mu).  `out` may hold preallocated (O, tO, lse, mu)."""
    lib = load()
    if out is None:
        O, tO = _like(Q), _like(Q)
        lse = torch.empty(Q.shape[:3], dtype=torch.float32, device=Q.device)
        mu = torch.empty_like(lse)
    else:
        O, tO, lse, mu = out
    _check_tensors(Q, (tQ, O, tO))
    _check_tensors(K, (V, tK, tV))
    p = _params(Q, scale, flags, K)
    with torch.cuda.device(Q.device):
        rc = lib.tvm_attn_jvp_fwd(ctypes.byref(p), Q.data_ptr(), K.data_ptr(), V.data_ptr(), tQ.data_ptr(),
                                  tK.data_ptr(), tV.data_ptr(), O.data_ptr(), tO.data_ptr(), lse.data_ptr(),
                                  mu.data_ptr(), None, 0, _stream_ptr(stream))
    if rc != 0:
        _raise("tvm_attn_jvp_fwd", rc)
    return O, tO, lse, mu


def tvm_attn_jvp_bwd(Q, K, V, tQ, tK, tV, O, tO, lse, mu, dO, dtO, scale=0.0, flags=0, out=None, workspace=None,
                     stream=None):
    """Backward: returns (dQ, dK, dV, dtQ, dtK, dtV).  `workspace` is a uint8 CUDA tensor of at least
    tvm_attn_jvp_workspace_bytes(...) bytes; one is allocated with torch when not given.
    dO or dtO may be None (a zero cotangent; dtO=None is the "detach JVP" setting).  With dtO=None the entries
    dtQ, dtK, dtV of `out` may be None too; tensors given there come back zero."""
    lib = load()
    p = _params(Q, scale, flags, K)
    need = int(lib.tvm_attn_jvp_workspace_bytes(ctypes.byref(p), 1))
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=Q.device)
    outs = out if out is not None else (_like(Q), _like(K), _like(K), _like(Q), _like(K), _like(K))
    _check_tensors(Q, tuple(t for t in (tQ, O, tO, dO, dtO, outs[0], outs[3]) if t is not None))
    _check_tensors(K, tuple(t for t in (V, tK, tV, outs[1], outs[2], outs[4], outs[5]) if t is not None))
    with torch.cuda.device(Q.device):
        rc = lib.tvm_attn_jvp_bwd(ctypes.byref(p), Q.data_ptr(), K.data_ptr(), V.data_ptr(), tQ.data_ptr(),
                                  tK.data_ptr(), tV.data_ptr(), O.data_ptr(), tO.data_ptr(), lse.data_ptr(),
                                  mu.data_ptr(), _ptr(dO), _ptr(dtO), *[_ptr(o) for o in outs],
                                  workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    if rc != 0:
        _raise("tvm_attn_jvp_bwd", rc)
    return outs


def tvm_attn_jvp_bwd_noalloc(Q, K, V, tQ, tK, tV, O, tO, lse, mu, dO, dtO, out, scale=0.0, flags=0, stream=None):
    """Backward for callers that cannot allocate: same result as tvm_attn_jvp_bwd, scratch inside the library.

    `out` must hold the six preallocated gradient tensors (dQ, dK, dV, dtQ, dtK, dtV): this wrapper, like the
    C entry point behind it, allocates nothing.  B*H*N may not exceed NOALLOC_MAX_ROWS.  Calls that may overlap
    on the GPU race on the shared scratch; the first call on a device should come before any stream capture."""
    lib = load()
    _check_tensors(Q, tuple(t for t in (tQ, O, tO, dO, dtO, out[0], out[3]) if t is not None))
    _check_tensors(K, tuple(t for t in (V, tK, tV, out[1], out[2], out[4], out[5]) if t is not None))
    p = _params(Q, scale, flags, K)
    with torch.cuda.device(Q.device):
        rc = lib.tvm_attn_jvp_bwd_noalloc(ctypes.byref(p), Q.data_ptr(), K.data_ptr(), V.data_ptr(), tQ.data_ptr(),
                                          tK.data_ptr(), tV.data_ptr(), O.data_ptr(), tO.data_ptr(), lse.data_ptr(),
                                          mu.data_ptr(), _ptr(dO), _ptr(dtO), *[_ptr(o) for o in out],
                                          _stream_ptr(stream))
    if rc != 0:
        _raise("tvm_attn_jvp_bwd_noalloc", rc)
    return tuple(out)


def _check_scale(g, ref):
    if g.dtype != torch.float32 or g.dim() != 1 or g.numel() != ref.shape[-1] or g.device != ref.device or not g.is_contiguous():
        raise ValueError("a scale must be a contiguous float32 CUDA vector of d elements")


def tvm_qk_rmsnorm_jvp_fwd(Q, tQ, K, tK, gQ, gK, eps=1e-6, stream=None):
    """RMSNorm QK-normalisation with a tangent: returns (Qn, tQn, Kn, tKn)."""
    lib = load()
    _check_tensors(Q, (tQ,))
    _check_tensors(K, (tK,))
    _check_scale(gQ, Q)
    _check_scale(gK, Q)
    p = _params(Q, 0.0, 0, K)
    outs = (_like(Q), _like(Q), _like(K), _like(K))
    with torch.cuda.device(Q.device):
        rc = lib.tvm_qk_rmsnorm_jvp_fwd(ctypes.byref(p), float(eps), Q.data_ptr(), tQ.data_ptr(), K.data_ptr(), tK.data_ptr(),
                                        gQ.data_ptr(), gK.data_ptr(), *[o.data_ptr() for o in outs], _stream_ptr(stream))
    if rc != 0:
        _raise("tvm_qk_rmsnorm_jvp_fwd", rc)
    return outs


def tvm_qk_rmsnorm_jvp_bwd(Q, tQ, K, tK, gQ, gK, dQn, dtQn, dKn, dtKn, eps=1e-6, workspace=None, stream=None):
    """Backward of the normalisation: returns (dQ, dtQ, dK, dtK, dgQ, dgK)."""
    lib = load()
    _check_tensors(Q, (tQ, dQn, dtQn))
    _check_tensors(K, (tK, dKn, dtKn))
    _check_scale(gQ, Q)
    _check_scale(gK, Q)
    p = _params(Q, 0.0, 0, K)
    need = int(lib.tvm_qk_rmsnorm_jvp_workspace_bytes(ctypes.byref(p)))
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=Q.device)
    outs = (_like(Q), _like(Q), _like(K), _like(K))
    dgQ, dgK = torch.empty_like(gQ), torch.empty_like(gK)
    with torch.cuda.device(Q.device):
        rc = lib.tvm_qk_rmsnorm_jvp_bwd(ctypes.byref(p), float(eps), Q.data_ptr(), tQ.data_ptr(), K.data_ptr(), tK.data_ptr(),
                                        gQ.data_ptr(), gK.data_ptr(), dQn.data_ptr(), dtQn.data_ptr(), dKn.data_ptr(),
                                        dtKn.data_ptr(), *[o.data_ptr() for o in outs], dgQ.data_ptr(), dgK.data_ptr(),
                                        workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    if rc != 0:
        _raise("tvm_qk_rmsnorm_jvp_bwd", rc)
    return outs + (dgQ, dgK)


def tvm_attn_check_status(stream=None, raise_on_error=True):
    rc = int(load().tvm_attn_check_status(_stream_ptr(stream)))
    if rc != 0 and raise_on_error:
        _raise("tvm_attn_check_status", rc)
    return rc


def tvm_attn_selftest_timeout(limit_ns=1_000_000, stream=None):
    """Enqueues the kernel whose bounded wait runs out on purpose (see include/tvm_attn.h)."""
    rc = int(load().tvm_attn_selftest_timeout(int(limit_ns), _stream_ptr(stream)))
    if rc != 0:
        _raise("tvm_attn_selftest_timeout", rc)


def tvm_attn_launch_count():
    return int(load().tvm_attn_launch_count())


def tvm_attn_version():
    return int(load().tvm_attn_version())


def tvm_attn_set_profiling(enable):
    load().tvm_attn_set_profiling(1 if enable else 0)


def tvm_attn_get_profile():
    """Per-kernel milliseconds of the most recent profiled call, in launch order."""
    buf = (ctypes.c_float * 8)()
    n = int(load().tvm_attn_get_profile(buf, 8))
    if n < 0:
        _raise("tvm_attn_get_profile", n)
    return [float(buf[k]) for k in range(n)]
