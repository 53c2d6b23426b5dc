"""Seeded synthetic inputs for the attention-JVP path.

This module holds no arithmetic of the method itself: it only draws the eight input tensors
(Q, K, V, their tangents tQ, tK, tV, and the cotangents dO, dtO) with the shapes and value
distributions of the workloads, so that the CUDA path and the CPU oracle can be fed the very
same numbers.  Shapes stand in for DiT-XL/2 attention layers on ImageNet-256/512 latents
(paper Sec. 5 and the experimental-settings table); no dataset is read.

Recipe: a torch CPU generator seeded per workload draws fp32 N(0,1) values in the fixed order
Q, K, V, tQ, tK, tV, dO, dtO; tangents are multiplied by 0.5; the "large" workload multiplies a
seeded 5 % of the rows of Q and of K (the same row indices per head in both) by 4 to make the
softmax peaky.  Callers round to bf16 themselves when they want the bf16 mode.
"""
import math
from collections import namedtuple

import torch

Workload = namedtuple("Workload", "name B H N d seed tangent_std peaky_frac")

WORKLOADS = {
    "tiny": Workload("tiny", 2, 2, 64, 32, 0, 1.0, 0.0),
    "dit256": Workload("dit256", 64, 16, 256, 72, 1, 0.5, 0.0),
    "dit512": Workload("dit512", 16, 16, 1024, 72, 2, 0.5, 0.0),
    "large": Workload("large", 2, 24, 4096, 128, 3, 0.5, 0.05),
}
for _n in (256, 1024, 4096, 16384, 32768):  # 32768: the longest sequence of the paper's kernel table (App. C)
    WORKLOADS["sweep%d" % _n] = Workload("sweep%d" % _n, max(1, 65536 // _n), 16, _n, 64, 4, 0.5, 0.0)

NAMES = ("Q", "K", "V", "tQ", "tK", "tV", "dO", "dtO")


def default_scale(d):
    """Softmax scale alpha = 1/sqrt(d) with the true head dimension."""
    return 1.0 / math.sqrt(d)


def custom(B, H, N, d, seed=0, tangent_std=0.5, peaky_frac=0.0):
    return Workload("custom", B, H, N, d, seed, tangent_std, peaky_frac)


def make_inputs(wl, heads=None):
    """Draws the eight (B, H, N, d) fp32 CPU tensors of a workload.

    heads: optional list of flat head indices (b*H + h); then only those heads are returned, as a
    (len(heads), 1, N, d) batch holding exactly the values the full tensors have at those heads.
    """
    if isinstance(wl, str):
        wl = WORKLOADS[wl]
    g = torch.Generator(device="cpu")
    g.manual_seed(1000 + wl.seed)
    shape = (wl.B, wl.H, wl.N, wl.d)
    out = {}
    for name in NAMES:
        x = torch.randn(shape, generator=g, dtype=torch.float32)
        if name in ("tQ", "tK", "tV") and wl.tangent_std != 1.0:
            x *= wl.tangent_std
        out[name] = x
    if wl.peaky_frac > 0.0:
        k = int(wl.peaky_frac * wl.N)
        if k > 0:
            scores = torch.rand((wl.B, wl.H, wl.N), generator=g)
            rows = scores.topk(k, dim=-1).indices  # k distinct row indices per head
            mult = torch.ones((wl.B, wl.H, wl.N, 1))
            mult.scatter_(2, rows.unsqueeze(-1), 4.0)
            out["Q"] *= mult
            out["K"] *= mult
    if heads is not None:
        idx = torch.as_tensor(list(heads), dtype=torch.long)
        for name in NAMES:
            out[name] = out[name].reshape(wl.B * wl.H, 1, wl.N, wl.d)[idx].contiguous()
    return out


def flops(B, H, N, d):
    """Analytic work of the path with the true d: 6 GEMMs forward, 15 GEMMs backward."""
    base = 2.0 * B * H * N * N * d
    return 6.0 * base, 15.0 * base
