"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB_DIR = os.path.join(_HERE, "_lib")
LIB_PATH = os.path.join(LIB_DIR, "libtvm_attn.so")
SOURCES = ["tvm_attn_api.cu"]


def _newest_source_mtime():
    newest = 0.0
    for d in (CSRC, os.path.join(_ROOT, "include")):
        for name in os.listdir(d):
            newest = max(newest, os.path.getmtime(os.path.join(d, name)))
    return newest


def nvcc_command(out_path, extra=()):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    return [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
            "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
            *extra, "-o", out_path, *[os.path.join(CSRC, s) for s in SOURCES]]


def build(force=False, verbose=False, out_path=None):
    """Compiles libtvm_attn.so if it is missing or older than its sources; returns its path.
    `out_path` writes the library somewhere else."""
    global_out = out_path or LIB_PATH
    if not force and os.path.exists(global_out) and os.path.getmtime(global_out) >= _newest_source_mtime():
        return global_out
    os.makedirs(os.path.dirname(global_out), exist_ok=True)
    tmp = global_out + ".tmp.%d" % os.getpid()
    extra = ("-Xptxas", "-v") if verbose else ()
    cmd = nvcc_command(tmp, extra)
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n%s\n%s" % (" ".join(cmd), res.stderr[-8000:]))
    if verbose:
        print(res.stderr)
    os.replace(tmp, global_out)
    return global_out


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
