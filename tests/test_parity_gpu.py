"""GPU parity: the CUDA path, called through the C-ABI binding, against the fp64 C oracle on the
same seeded inputs.  Error metric per tensor: max|gpu - ref| / max|ref|.

Tolerances: bf16 mode 1e-2 for O and tO, 2e-2 for the six gradients (inputs are rounded to bf16
once and the oracle consumes those rounded values, so only the kernels' own rounding counts);
fp32 validation mode 1e-4 for everything.  The saved statistics lse and mu are fp32 in both modes;
in bf16 mode they are held to 1e-4 as well: they are fp32 sums of exact products of the bf16 inputs, and only
mu passes through one more rounding (the exponentials that weight it).
"""
import threading

import numpy as np
import pytest
import torch

from paper_2511_19797_b200 import binding, inputs
from tests._parity import assert_within, run_case

pytestmark = pytest.mark.gpu

BF16_FWD, BF16_BWD, BF16_STATS, FP32_TOL = 1e-2, 2e-2, 1e-4, 1e-4


def test_tiny_fp32_validation_mode():
    errs, _, _ = run_case("tiny", dtype=torch.float32)
    assert_within(errs, FP32_TOL, FP32_TOL)


def test_tiny_bf16_tensor_cores():
    errs, _, _ = run_case("tiny")
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


def test_tiny_bf16_cuda_cores():
    errs, _, _ = run_case("tiny", flags=binding.FLAG_CUDA_CORES)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


@pytest.mark.parametrize("name,heads", [
    ("dit256", [0, 341, 682, 1023]),
    ("dit512", [0, 85, 170, 255]),
    ("large", [0, 47]),
    ("sweep256", [0, 1365, 2730, 4095]),
    ("sweep1024", [0, 341, 682, 1023]),
    ("sweep4096", [0, 255]),
])
def test_full_size_workloads_on_sampled_heads(name, heads):
    errs, _, _ = run_case(name, oracle_heads=heads)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


@pytest.mark.parametrize("B,H,N,d", [
    (1, 1, 1, 8), (1, 2, 7, 16), (2, 1, 64, 64), (1, 1, 100, 72), (1, 3, 129, 40), (2, 2, 191, 128),
    (1, 1, 257, 72), (1, 2, 320, 32), (1, 1, 1000, 24), (1, 2, 130, 80), (2, 1, 96, 56), (1, 1, 66, 104),
])
@pytest.mark.parametrize("mode", ["bf16", "fp32"])
def test_ragged_and_degenerate_shapes(B, H, N, d, mode):
    wl = inputs.custom(B, H, N, d, seed=100 + N + d)
    if mode == "fp32":
        errs, _, _ = run_case(wl, dtype=torch.float32)
        assert_within(errs, FP32_TOL, FP32_TOL)
    else:
        errs, _, _ = run_case(wl)
        assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


@pytest.mark.parametrize("B,H,N,d", [(3, 50, 192, 72), (3, 50, 320, 64), (5, 61, 65, 72), (2, 80, 200, 40),
                                     (4, 50, 64, 72), (4, 50, 33, 40)])
def test_several_work_items_per_cta(B, H, N, d):
    """More work items than SMs (one CTA per SM walks through several of them), with odd numbers of stream
    tiles per item (3, 5, 2, 4, 1, 1 tiles of 64), so that buffer and barrier parities differ from item to item,
    and a ragged last tile."""
    wl = inputs.custom(B, H, N, d, seed=300 + N + d)
    errs, _, _ = run_case(wl)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


@pytest.mark.parametrize("B,H,N,d", [
    (1, 108, 129, 80), (1, 173, 383, 72), (1, 559, 16, 8), (2, 17, 640, 40), (2, 210, 65, 72), (2, 95, 383, 64),
    (3, 116, 65, 80), (3, 43, 384, 80), (3, 27, 640, 64), (5, 102, 31, 56), (5, 16, 250, 48), (5, 40, 128, 64),
])
def test_many_heads_of_odd_shapes_on_sampled_heads(B, H, N, d):
    """Shapes drawn at random (sequence lengths around the tile boundaries, every padded head dim), each with
    more work items than SMs; the oracle runs on a dozen sampled heads."""
    wl = inputs.custom(B, H, N, d, seed=1000 + N + d)
    heads = sorted(set(int(i) for i in np.random.default_rng(N * 131 + d).integers(0, B * H, 12)))
    errs, _, _ = run_case(wl, oracle_heads=heads)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


def test_explicit_scale_is_honoured():
    wl = inputs.custom(1, 2, 96, 48, seed=7)
    errs, _, _ = run_case(wl, scale=0.05)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


@pytest.mark.parametrize("N,d", [(200, 72), (129, 72), (65, 64)])
def test_runs_are_bit_reproducible_and_respect_buffer_bounds(N, d):
    # (an odd number of rows: the last row has no partner in the pass that writes its outputs by lane pairs)
    wl = inputs.custom(2, 2, N, d, seed=9)
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()}
    n = x["Q"].numel()

    def padded():
        buf = torch.full((n + 512,), 123.0, dtype=torch.bfloat16, device="cuda")
        return buf, buf[256:256 + n].view_as(x["Q"])

    runs = []
    for _ in range(2):
        bufs = [padded() for _ in range(8)]
        lse = torch.empty(x["Q"].shape[:3], dtype=torch.float32, device="cuda")
        mu = torch.empty_like(lse)
        O, tO, lse, mu = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"],
                                                  out=(bufs[0][1], bufs[1][1], lse, mu))
        grads = binding.tvm_attn_jvp_bwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], O, tO, lse, mu, x["dO"],
                                         x["dtO"], out=tuple(b[1] for b in bufs[2:]))
        binding.tvm_attn_check_status()
        for full, _ in bufs:
            assert torch.all(full[:256] == 123.0) and torch.all(full[256 + n:] == 123.0), "wrote outside a buffer"
        runs.append([t.clone() for t in (O, tO, lse, mu) + tuple(grads)])
    for a, b in zip(*runs):
        assert torch.equal(a, b)


def test_calls_replay_from_a_cuda_graph():
    """Forward and backward recorded by stream capture and replayed give, bit for bit, what the direct calls gave."""
    wl = inputs.custom(2, 4, 320, 72, seed=21)
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()}
    q = x["Q"]
    outs = [torch.empty_like(q), torch.empty_like(q), torch.empty(q.shape[:3], dtype=torch.float32, device="cuda"),
            torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")] + [torch.empty_like(q) for _ in range(6)]
    ws = torch.empty(binding.tvm_attn_jvp_workspace_bytes(*q.shape), dtype=torch.uint8, device="cuda")

    def step():
        binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], out=tuple(outs[:4]))
        binding.tvm_attn_jvp_bwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], outs[0], outs[1], outs[2], outs[3],
                                 x["dO"], x["dtO"], out=tuple(outs[4:]), workspace=ws)

    step()
    binding.tvm_attn_check_status()
    want = [t.clone() for t in outs]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for _ in range(2):
        for t in outs:
            t.zero_()
        graph.replay()
        binding.tvm_attn_check_status()
        for a, b in zip(outs, want):
            assert torch.equal(a, b)


def test_errors_reported_on_the_gpu_box():
    x = torch.zeros(1, 1, 64, 36, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.TvmAttnError) as e:
        binding.tvm_attn_jvp_fwd(x, x, x, x, x, x)
    assert e.value.code == -2
    y = torch.zeros(1, 1, 64, 32, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(1, 1, 64, device="cuda")
    with pytest.raises(binding.TvmAttnError) as e:
        binding.tvm_attn_jvp_bwd(y, y, y, y, y, y, y, y, lse, lse, y, y,
                                 workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
    assert binding.tvm_attn_launch_count() >= 0


def test_longest_sequence_whole_heads():
    """The longest sweep point as it is benchmarked (B=4, H=16, N=16384, d=64: 8192 work items of 256 stream
    tiles each, dozens per CTA), all ten outputs element by element on four whole heads.  The C oracle takes a
    few minutes per head on one core; the four heads run on four threads."""
    errs, _, _ = run_case("sweep16384", oracle_heads=[0, 21, 42, 63])
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


def test_longest_sequence_on_sampled_query_rows():
    """N = 16384 on a reduced batch, query-side outputs on sampled rows against the whole-matrix numpy oracle
    (which accepts fewer query rows than keys): a second, independent writing of the definitions at this length."""
    from oracle import attn_jvp_numpy as onp
    wl = inputs.custom(1, 2, 16384, 64, seed=4, tangent_std=0.5)
    x = {k: v.to(torch.bfloat16) for k, v in inputs.make_inputs(wl).items()}
    dev = {k: v.cuda() for k, v in x.items()}
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"])
    grads = binding.tvm_attn_jvp_bwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], O, tO, lse, mu,
                                     dev["dO"], dev["dtO"])
    binding.tvm_attn_check_status()
    rows = [0, 1, 127, 128, 5000, 8191, 12345, 16383]
    f64 = {k: v.to(torch.float64).numpy() for k, v in x.items()}
    sub = lambda k: np.ascontiguousarray(f64[k][:, :, rows])
    alpha = inputs.default_scale(64)
    rO, rtO, rlse, rmu = onp.attn_jvp_fwd(sub("Q"), f64["K"], f64["V"], sub("tQ"), f64["tK"], f64["tV"], alpha)
    rdQ, _, _, rdtQ, _, _ = onp.attn_jvp_bwd(sub("Q"), f64["K"], f64["V"], sub("tQ"), f64["tK"], f64["tV"], sub("dO"),
                                             sub("dtO"), alpha)
    pick = lambda t: t.float().cpu().numpy()[:, :, rows]
    from tests._parity import rel_err
    errs = {"O": rel_err(pick(O), rO), "tO": rel_err(pick(tO), rtO), "lse": rel_err(pick(lse), rlse),
            "mu": rel_err(pick(mu), rmu), "dQ": rel_err(pick(grads[0]), rdQ), "dtQ": rel_err(pick(grads[3]), rdtQ)}
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


def test_gradients_are_complete_for_work_enqueued_behind_the_call():
    """The three tensor-core passes of one backward call overlap (the later ones start while the earlier ones
    drain).  Work enqueued on the same stream right after the call, with no host synchronisation in between,
    must still see all six gradients complete."""
    wl = inputs.custom(4, 37, 320, 72, seed=77)          # one wave is not enough: the passes do overlap
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()}
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"])
    args = (x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], O, tO, lse, mu, x["dO"], x["dtO"])
    for _ in range(3):
        out = tuple(torch.full_like(x["Q"], float("nan")) for _ in range(6))
        torch.cuda.synchronize()
        binding.tvm_attn_jvp_bwd(*args, out=out)
        seen = [t.clone() for t in out]                   # consumer kernels on the same stream, no sync before them
        torch.cuda.synchronize()
        binding.tvm_attn_check_status()
        for name, a, b in zip(("dQ", "dK", "dV", "dtQ", "dtK", "dtV"), seen, out):
            assert torch.isfinite(a.float()).all(), name
            assert torch.equal(a, b), name


def test_bounded_wait_that_runs_out_is_reported_and_later_kernels_are_no_ops():
    """Failure reporting, exercised without disturbing a real kernel: a one-warp kernel waits (1 ms limit) on a
    barrier nobody signals, gives up and raises the device status.  A forward enqueued behind it must not touch
    its outputs; the status is reported once and cleared; the next forward works."""
    wl = inputs.custom(1, 2, 200, 72, seed=12)
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()}
    ref = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"])
    assert binding.tvm_attn_check_status(raise_on_error=False) == 0
    O, tO = torch.full_like(x["Q"], 7.0), torch.full_like(x["Q"], 7.0)
    lse = torch.full(x["Q"].shape[:3], 7.0, device="cuda")
    mu = torch.full_like(lse, 7.0)
    binding.tvm_attn_selftest_timeout(1_000_000)
    binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], out=(O, tO, lse, mu))
    assert binding.tvm_attn_check_status(raise_on_error=False) == -5          # DEVICE_TIMEOUT
    for t in (O, tO, lse, mu):
        assert torch.all(t == 7.0), "a kernel behind the time-out wrote its outputs"
    assert binding.tvm_attn_check_status(raise_on_error=False) == 0           # reported once, then cleared
    with pytest.raises(binding.TvmAttnError):
        binding.tvm_attn_selftest_timeout(0)
    got = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], out=(O, tO, lse, mu))
    binding.tvm_attn_check_status()
    for a, b in zip(got, ref):
        assert torch.equal(a, b)


def test_two_host_threads_on_two_streams():
    """Concurrent calls from two host threads, each on its own stream with its own buffers and workspace, give
    the results of the same calls made one after the other."""
    wls = [inputs.custom(2, 9, 260, 72, seed=41), inputs.custom(3, 5, 200, 64, seed=42)]
    xs = [{k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()} for wl in wls]

    def run(x, stream):
        with torch.cuda.stream(stream):
            fw = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], stream=stream)
            gr = binding.tvm_attn_jvp_bwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], *fw, x["dO"], x["dtO"],
                                          stream=stream)
        return tuple(fw) + tuple(gr)

    serial = [run(x, torch.cuda.current_stream()) for x in xs]
    torch.cuda.synchronize()
    results, errors = [None, None], []

    def worker(i):
        try:
            st = torch.cuda.Stream()
            for _ in range(5):
                results[i] = run(xs[i], st)
            st.synchronize()
        except Exception as e:  # noqa: BLE001
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    binding.tvm_attn_check_status()
    for i in range(2):
        for a, b in zip(results[i], serial[i]):
            assert torch.equal(a, b)


def _sampled_query_rows(N, rows, seed):
    """Query-side outputs of a B=1, H=2, d=64 problem with N keys on sampled query rows against the numpy oracle."""
    from oracle import attn_jvp_numpy as onp
    from tests._parity import rel_err
    wl = inputs.custom(1, 2, N, 64, seed=seed, tangent_std=0.5)
    x = {k: v.to(torch.bfloat16) for k, v in inputs.make_inputs(wl).items()}
    dev = {k: v.cuda() for k, v in x.items()}
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"])
    grads = binding.tvm_attn_jvp_bwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], O, tO, lse, mu,
                                     dev["dO"], dev["dtO"])
    binding.tvm_attn_check_status()
    f64 = {k: v.to(torch.float64).numpy() for k, v in x.items()}
    sub = lambda k: np.ascontiguousarray(f64[k][:, :, rows])
    alpha = inputs.default_scale(64)
    rO, rtO, rlse, rmu = onp.attn_jvp_fwd(sub("Q"), f64["K"], f64["V"], sub("tQ"), f64["tK"], f64["tV"], alpha)
    rdQ, _, _, rdtQ, _, _ = onp.attn_jvp_bwd(sub("Q"), f64["K"], f64["V"], sub("tQ"), f64["tK"], f64["tV"], sub("dO"),
                                             sub("dtO"), alpha)
    pick = lambda t: t.float().cpu().numpy()[:, :, rows]
    return {"O": rel_err(pick(O), rO), "tO": rel_err(pick(tO), rtO), "lse": rel_err(pick(lse), rlse),
            "mu": rel_err(pick(mu), rmu), "dQ": rel_err(pick(grads[0]), rdQ), "dtQ": rel_err(pick(grads[3]), rdtQ)}


def test_sequence_of_32768_query_side_on_sampled_rows():
    """The longest sequence of the paper's kernel table (App. C, S = 32,768) on one GPU: O, tO, lse, mu, dQ, dtQ
    on sampled query rows."""
    errs = _sampled_query_rows(32768, [0, 127, 128, 9999, 16384, 20000, 32767], seed=6)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


def test_sequence_of_32768_key_side_with_cotangents_on_few_rows():
    """Key-side gradients at S = 32,768, every element of them: the cotangents are non-zero on 48 query rows only,
    so only those rows contribute to dK, dtK, dV, dtV and the whole-matrix numpy oracle can compute them from the
    48 rows against all 32,768 keys, while the GPU runs the full problem.  Query rows with a zero cotangent must
    come out with exactly zero dQ and dtQ."""
    from oracle import attn_jvp_numpy as onp
    from tests._parity import rel_err
    N = 32768
    wl = inputs.custom(1, 2, N, 64, seed=8, tangent_std=0.5)
    x = {k: v.to(torch.bfloat16) for k, v in inputs.make_inputs(wl).items()}
    rows = sorted(set(int(i) for i in np.random.default_rng(5).integers(0, N, 48)) | {0, 63, 64, N - 1})
    mask = torch.zeros(1, 1, N, 1, dtype=torch.bfloat16)
    mask[:, :, rows] = 1
    x["dO"] = x["dO"] * mask
    x["dtO"] = x["dtO"] * mask
    dev = {k: v.cuda() for k, v in x.items()}
    O, tO, lse, mu = binding.tvm_attn_jvp_fwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"])
    dQ, dK, dV, dtQ, dtK, dtV = binding.tvm_attn_jvp_bwd(dev["Q"], dev["K"], dev["V"], dev["tQ"], dev["tK"], dev["tV"], O, tO,
                                                         lse, mu, dev["dO"], dev["dtO"])
    binding.tvm_attn_check_status()
    f64 = {k: v.to(torch.float64).numpy() for k, v in x.items()}
    sub = lambda k: np.ascontiguousarray(f64[k][:, :, rows])
    alpha = inputs.default_scale(64)
    rdQ, rdK, rdV, rdtQ, rdtK, rdtV = onp.attn_jvp_bwd(sub("Q"), f64["K"], f64["V"], sub("tQ"), f64["tK"], f64["tV"],
                                                       sub("dO"), sub("dtO"), alpha)
    f = lambda t: t.float().cpu().numpy()
    errs = {"dK": rel_err(f(dK), rdK), "dtK": rel_err(f(dtK), rdtK), "dV": rel_err(f(dV), rdV), "dtV": rel_err(f(dtV), rdtV),
            "dQ": rel_err(f(dQ)[:, :, rows], rdQ), "dtQ": rel_err(f(dtQ)[:, :, rows], rdtQ)}
    assert_within(errs, BF16_FWD, BF16_BWD)
    others = np.setdiff1d(np.arange(N), rows)
    assert not f(dQ)[:, :, others].any() and not f(dtQ)[:, :, others].any()


ABSENT_SHAPES = [(2, 3, 200, 72), (1, 2, 129, 64), (3, 50, 192, 72), (1, 4, 333, 40), (2, 2, 64, 80)]


@pytest.mark.parametrize("absent", ["dtO", "dO"])
@pytest.mark.parametrize("B,H,N,d", ABSENT_SHAPES)
def test_absent_cotangent_counts_as_zero(absent, B, H, N, d):
    """A null dO or dtO (Sec. 5.3 "detach JVP": no gradient through tO) against the oracle fed a zero cotangent."""
    wl = inputs.custom(B, H, N, d, seed=500 + N + d)
    heads = None if B * H <= 12 else [0, 7, 77, B * H - 1]
    errs, got, _ = run_case(wl, oracle_heads=heads, absent=absent)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)
    if absent == "dtO":
        for k in ("dtQ", "dtK", "dtV"):
            assert not got[k].any(), k


@pytest.mark.parametrize("absent", ["dtO", "dO"])
def test_absent_cotangent_on_the_headline_shape(absent):
    errs, _, _ = run_case("dit512", oracle_heads=[0, 85, 255], absent=absent)
    assert_within(errs, BF16_FWD, BF16_BWD, BF16_STATS)


@pytest.mark.parametrize("absent", ["dtO", "dO"])
def test_absent_cotangent_fp32_validation_mode(absent):
    errs, _, _ = run_case("tiny", dtype=torch.float32, absent=absent)
    assert_within(errs, FP32_TOL, FP32_TOL)


def test_detached_backward_needs_no_tangent_gradient_buffers():
    """With dtO absent the outputs dtQ, dtK, dtV may be null; dQ, dK, dV are those of the call that is given them."""
    wl = inputs.custom(2, 2, 200, 72, seed=21)
    x = {k: v.to(torch.bfloat16).cuda() for k, v in inputs.make_inputs(wl).items()}
    fw = binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"])
    args = (x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"]) + tuple(fw)
    full = binding.tvm_attn_jvp_bwd(*args, x["dO"], None)
    three = tuple(torch.empty_like(x["Q"]) for _ in range(3)) + (None, None, None)
    part = binding.tvm_attn_jvp_bwd(*args, x["dO"], None, out=three)
    binding.tvm_attn_check_status()
    for a, b in zip(part[:3], full[:3]):
        assert torch.equal(a, b)
    with pytest.raises(binding.TvmAttnError) as e:        # both cotangents absent: nothing to differentiate
        binding.tvm_attn_jvp_bwd(*args, None, None)
    assert e.value.code == -1
    with pytest.raises(binding.TvmAttnError) as e:        # dtO given: its gradients need somewhere to go
        binding.tvm_attn_jvp_bwd(*args, x["dO"], x["dtO"], out=three)
    assert e.value.code == -1
