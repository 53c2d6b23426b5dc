#!/usr/bin/env python
"""Benchmark of the fused attention-JVP forward + backward path on B200.

One "step" is one forward call plus one backward call of the C-ABI library over one batch of
synthetic DiT-shaped input (default workload: B=16, H=16, N=1024, d=72, bf16).  The metric is
TFLOP/s with the analytic work of the method (12*B*H*N^2*d forward, 30*B*H*N^2*d backward, true d).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line.  Under torchrun every rank runs the same per-GPU workload on its own GPU
(heads are independent, no collective in the data path: weak scaling); rank 0 prints.
`--impl reference` times the fp64 CPU oracle on the host cores instead (a baseline, not a target).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "attn_jvp_fwd_bwd_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# GEMM units (2*B*H*N^2*d FLOP each, true d) each kernel EXECUTES by design.  The backward passes recompute
# scores: together they execute 24 units for the 15 the method counts (3 recompute + 3 cotangent-score + 9 output).
KERNEL_GEMMS = {"fwd": 6, "bwd_rowsums": 0, "bwd_dv": 6, "bwd_dk": 9, "bwd_dq": 9}
BWD_CREDITED_GEMMS = 15
BWD_TC = ("bwd_dv", "bwd_dk", "bwd_dq")
# (B,H,N,d) tensors each kernel reads + writes once (its algorithmic HBM bytes, in units of one tensor)
KERNEL_TENSORS = {"fwd": 8, "bwd_rowsums": 4, "bwd_dv": 8, "bwd_dk": 10, "bwd_dq": 10}
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in
# profiles/jvp_fwd_bwd_kernels_dit512.md (that workload only; None for anything else, and None once a kernel
# has changed since the capture)
NCU_TRAFFIC_BYTES = {"dit512": {"fwd": 280.0e6, "bwd_dv": 281.5e6, "bwd_dk": 366.3e6, "bwd_dq": 363.7e6}}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            pk = json.load(f)
        return {k: float(pk[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def wait_first(self, timeout=5.0):
        """Blocks until nvidia-smi has delivered its first sample (it takes a moment to start)."""
        t0 = time.time()
        while self.proc is not None and not self.rows and time.time() - t0 < timeout:
            time.sleep(0.02)

    def mark(self):
        """Samples taken before this call are dropped: only the timed region is summarised."""
        self.rows = []

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(wl_name, target_seconds=12.0, threads=None, heads=None):
    """Times the C oracle (forward + backward) on a bounded sample of whole heads of the workload.
    Returns (TFLOP/s, threads, description, seconds)."""
    import numpy as np
    import torch
    from oracle import c_oracle
    from paper_2511_19797_b200 import inputs
    wl = inputs.WORKLOADS[wl_name]
    cores = threads or c_oracle.default_threads()
    f_fwd, f_bwd = inputs.flops(1, 1, wl.N, wl.d)
    alpha = inputs.default_scale(wl.d)
    if heads is None:
        heads = calibrate_heads(wl, cores, alpha, target_seconds)
    idx = [int(i) for i in np.linspace(0, wl.B * wl.H - 1, heads).round()]
    x = inputs.make_inputs(wl, heads=idx)
    xs = [x[k].to(torch.bfloat16).to(torch.float64).numpy() for k in inputs.NAMES]
    t0 = time.perf_counter()
    used = c_oracle.attn_jvp_fwd(*xs[:6], alpha, nthreads=cores)[4]
    c_oracle.attn_jvp_bwd(*xs, alpha, nthreads=cores)
    dt = time.perf_counter() - t0
    tflops = heads * (f_fwd + f_bwd) / dt / 1e12
    desc = "%d of %d heads of %s (fwd+bwd, fp64 C oracle, gcc -O2), %.1f s" % (heads, wl.B * wl.H, wl_name, dt)
    return tflops, used, desc, dt, heads


def calibrate_heads(wl, cores, alpha, target_seconds):
    """Times one head per thread and returns how many whole heads make about `target_seconds` of CPU work."""
    import torch
    from oracle import c_oracle
    from paper_2511_19797_b200 import inputs
    probe = min(cores, wl.B * wl.H)
    xp = inputs.make_inputs(wl, heads=list(range(probe)))
    xps = [xp[k].to(torch.bfloat16).to(torch.float64).numpy() for k in inputs.NAMES]
    t0 = time.perf_counter()
    c_oracle.attn_jvp_fwd(*xps[:6], alpha, nthreads=cores)
    c_oracle.attn_jvp_bwd(*xps, alpha, nthreads=cores)
    t_probe = max(time.perf_counter() - t0, 1e-3)
    heads = int(max(1, min(wl.B * wl.H, round(probe * target_seconds / t_probe))))
    if heads >= cores:
        heads = max(cores, heads // cores * cores)
    return heads


def run_reference(args, rank):
    if rank != 0:
        return
    from paper_2511_19797_b200 import inputs
    wl = inputs.WORKLOADS[args.workload]
    times, vals = [], []
    # each step is a bounded sample; the whole run stays within a few minutes whatever K and W are
    per_step = max(0.25, min(6.0, 150.0 / max(1, args.warmup + args.steps)))
    heads = None
    for it in range(args.warmup + args.steps):
        v, cores, desc, dt, heads = oracle_sample(args.workload, target_seconds=per_step, heads=heads)
        if it >= args.warmup:
            times.append(dt); vals.append(v)
    value = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(times), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "B": wl.B, "H": wl.H, "N": wl.N, "d": wl.d,
                   "note": "each step is a bounded sample of whole heads of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="dit512")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default="full", choices=["full", "detach"],
                    help="detach: backward without dtO (no gradient through tO; Sec. 5.3 'detach JVP'), 10*B*H*N^2*d FLOP")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--max-regions", type=int, default=64, help="upper limit of repeated timed regions (1 for profiler runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2511_19797_b200 import binding, inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.load()

    wl = inputs.WORKLOADS[args.workload]
    f_fwd, f_bwd = inputs.flops(wl.B, wl.H, wl.N, wl.d)
    detach = args.variant == "detach"
    if detach:  # standard attention backward: S recompute, dP, dV, dK, dQ = 5 GEMM units
        f_bwd = f_bwd * 5.0 / 15.0
        KERNEL_GEMMS.update({"bwd_dv": 4, "bwd_dk": 6, "bwd_dq": 7})   # what the three passes still execute
        KERNEL_TENSORS.update({"bwd_rowsums": 2, "bwd_dv": 6, "bwd_dk": 8, "bwd_dq": 8})
    host = {k: v.to(torch.bfloat16).pin_memory() for k, v in inputs.make_inputs(wl).items()}
    x = {k: v.to(dev) for k, v in host.items()}
    shape = x["Q"].shape
    O, tO = torch.empty_like(x["Q"]), torch.empty_like(x["Q"])
    lse = torch.empty(shape[:3], dtype=torch.float32, device=dev)
    mu = torch.empty_like(lse)
    grads = tuple(torch.empty_like(x["Q"]) for _ in range(6))
    ws = torch.empty(max(16, binding.tvm_attn_jvp_workspace_bytes(*shape)), dtype=torch.uint8, device=dev)

    def fwd():
        binding.tvm_attn_jvp_fwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], out=(O, tO, lse, mu))

    def bwd():
        if detach:
            binding.tvm_attn_jvp_bwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], O, tO, lse, mu, x["dO"], None,
                                     out=grads[:3] + (None, None, None), workspace=ws)
        else:
            binding.tvm_attn_jvp_bwd(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], O, tO, lse, mu, x["dO"], x["dtO"],
                                     out=grads, workspace=ws)

    def step():
        fwd()
        bwd()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, n):
        """n back-to-back calls between CUDA events on torch's current stream (the one the library is given)."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    for _ in range(args.warmup):
        step()
    binding.tvm_attn_check_status()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_first()
        sampler.mark()
    # The timed region is exactly `steps` steps between two events.  A short region (20 steps are 30 ms) gives the
    # clock sampler a single sample, so the same region is measured `repeats` times in a row, until about half a
    # second has passed, and the median region is reported; every region keeps its own barrier + synchronise.
    launches0 = binding.tvm_attn_launch_count()
    regions = [timed(step, args.steps)]
    launches = binding.tvm_attn_launch_count() - launches0
    budget_ms = 500.0
    while sum(regions) < budget_ms and len(regions) < args.max_regions:
        regions.append(timed(step, args.steps))
    ms_total = statistics.median(regions)
    ms_fwd = statistics.median([timed(fwd, args.steps) for _ in range(max(1, min(len(regions), 16)))])
    ms_bwd = statistics.median([timed(bwd, args.steps) for _ in range(max(1, min(len(regions), 16)))])
    clocks = sampler.stop() if rank == 0 else None
    binding.tvm_attn_check_status()

    # per-kernel durations (CUDA events recorded by the library around each launch)
    binding.tvm_attn_set_profiling(True)
    per_kernel = {k: [] for k in KERNEL_GEMMS}
    for _ in range(min(args.steps, 20)):
        fwd()
        per_kernel["fwd"].append(binding.tvm_attn_get_profile()[0])
        bwd()
        prof = binding.tvm_attn_get_profile()
        for k, v in zip(("bwd_rowsums", "bwd_dv", "bwd_dk", "bwd_dq"), prof):
            per_kernel[k].append(v)
    binding.tvm_attn_set_profiling(False)
    kernel_ms = {k: statistics.mean(v) for k, v in per_kernel.items() if v}

    # end to end: pinned host inputs -> device, forward + backward, results -> pinned host
    out_names = ("O", "tO", "dQ", "dK", "dV") + (() if detach else ("dtQ", "dtK", "dtV"))
    in_names = tuple(k for k in inputs.NAMES if not (detach and k == "dtO"))
    host_out = {k: torch.empty(shape, dtype=torch.bfloat16).pin_memory() for k in out_names}
    host_stats = {k: torch.empty(shape[:3], dtype=torch.float32).pin_memory() for k in ("lse", "mu")}

    # The batch is cut into chunks (heads are independent) and the three legs run on three streams: while chunk c is
    # computed, chunk c + 1 comes in and chunk c - 1 goes out.  Events order the legs within a step and across steps
    # (a chunk's device buffers are rewritten by the next step).
    n_chunks = 4 if wl.B % 4 == 0 else 1
    cb = wl.B // n_chunks
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(n_chunks)]
    ev_comp = [torch.cuda.Event() for _ in range(n_chunks)]
    ev_out = [torch.cuda.Event() for _ in range(n_chunks)]
    ws_c = torch.empty(binding.tvm_attn_jvp_workspace_bytes(cb, wl.H, wl.N, wl.d), dtype=torch.uint8, device=dev)
    started = [False]

    def e2e_step():
        comp = torch.cuda.current_stream()
        for c in range(n_chunks):
            sl = slice(c * cb, (c + 1) * cb)
            if started[0]:
                s_in.wait_event(ev_comp[c])     # the step before has consumed this chunk's inputs
            with torch.cuda.stream(s_in):
                for k in in_names:
                    x[k][sl].copy_(host[k][sl], non_blocking=True)
                ev_in[c].record(s_in)
            comp.wait_event(ev_in[c])
            if started[0]:
                comp.wait_event(ev_out[c])      # the step before has copied this chunk's results out
            binding.tvm_attn_jvp_fwd(x["Q"][sl], x["K"][sl], x["V"][sl], x["tQ"][sl], x["tK"][sl], x["tV"][sl],
                                     out=(O[sl], tO[sl], lse[sl], mu[sl]))
            g = tuple(t[sl] for t in grads)
            binding.tvm_attn_jvp_bwd(x["Q"][sl], x["K"][sl], x["V"][sl], x["tQ"][sl], x["tK"][sl], x["tV"][sl], O[sl], tO[sl],
                                     lse[sl], mu[sl], x["dO"][sl], None if detach else x["dtO"][sl],
                                     out=(g[:3] + (None, None, None)) if detach else g, workspace=ws_c)
            ev_comp[c].record(comp)
            s_out.wait_event(ev_comp[c])
            with torch.cuda.stream(s_out):
                for k, t in zip(out_names, (O, tO) + grads):
                    host_out[k][sl].copy_(t[sl], non_blocking=True)
                host_stats["lse"][sl].copy_(lse[sl], non_blocking=True)
                host_stats["mu"][sl].copy_(mu[sl], non_blocking=True)
                ev_out[c].record(s_out)
        comp.wait_event(ev_out[n_chunks - 1])   # the step ends when its last results are on the host
        started[0] = True

    if args.e2e_steps > 0:
        e2e_step()
        ms_e2e = timed(e2e_step, args.e2e_steps) / args.e2e_steps
    else:
        ms_e2e = None
    h2d = sum(host[k].numel() * 2 for k in in_names)
    d2h = sum(t.numel() * 2 for t in host_out.values()) + sum(t.numel() * 4 for t in host_stats.values())
    binding.tvm_attn_check_status()

    # The RMSNorm QK-normalisation prologue on the same shape (memory-bound; not part of the timed step)
    rms = None
    try:
        gq = torch.ones(wl.d, device=dev)
        ws_n = torch.empty(max(16, 2 * 592 * wl.d * 4), dtype=torch.uint8, device=dev)

        def nfwd():
            binding.tvm_qk_rmsnorm_jvp_fwd(x["Q"], x["tQ"], x["K"], x["tK"], gq, gq)

        def nbwd():
            binding.tvm_qk_rmsnorm_jvp_bwd(x["Q"], x["tQ"], x["K"], x["tK"], gq, gq, x["dO"], x["dtO"], x["V"], x["tV"], workspace=ws_n)

        for fn in (nfwd, nbwd):
            fn(); fn(); fn()
        rms = (timed(nfwd, 20) / 20, timed(nbwd, 20) / 20)
    except binding.TvmAttnError:
        rms = None

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_src = load_peaks()
    ms_step = ms_total / args.steps
    value = world * (f_fwd + f_bwd) / (ms_step * 1e-3) / 1e12
    fwd_tf = f_fwd / (ms_fwd / args.steps * 1e-3) / 1e12
    bwd_tf = f_bwd / (ms_bwd / args.steps * 1e-3) / 1e12
    unit_flops = 2.0 * wl.B * wl.H * wl.N * wl.N * wl.d
    tensor_bytes = 2.0 * wl.B * wl.H * wl.N * wl.d
    total_k = sum(kernel_ms.values())
    sm_mhz = (clocks or {}).get("sm_mhz")
    sm_max = (clocks or {}).get("sm_max_mhz")
    # Which measured peak the fractions are taken against: the burst figure when the GPU ran at (nearly) its
    # maximum clock through the timed regions or they were short, the sustained one when it ran power-capped.
    at_max_clock = bool(sm_mhz and sm_max and sm_mhz >= 0.97 * sm_max)
    short_run = sum(regions) < 1000.0
    use_burst = at_max_clock or (short_run and not sm_mhz)
    peak = peaks["bf16_tflops"] if use_burst else peaks["bf16_tflops_sustained"]
    peak_note = "%s %s bf16 GEMM peak: median SM clock %s of %s MHz over %d timed regions (%.0f ms)" % (
        peak_src, "burst" if use_burst else "sustained", sm_mhz, sm_max, len(regions), sum(regions))

    def cycles(ms):  # device time in SM clocks at the sampled median clock: comparable between short and long runs
        return None if not sm_mhz else ms * 1e-3 * sm_mhz * 1e6

    def fracs(tf):
        return {"frac_of_burst_peak": tf / peaks["bf16_tflops"], "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"],
                "frac_of_nominal": tf / NOMINAL_BF16_TFLOPS}

    # the dominant kernels: the three tensor-core passes of the backward, taken together
    tc_ms = sum(kernel_ms[k] for k in BWD_TC)
    credited_units = 5 if detach else BWD_CREDITED_GEMMS
    credited = credited_units * unit_flops / (tc_ms * 1e-3) / 1e12
    executed = sum(KERNEL_GEMMS[k] for k in BWD_TC) * unit_flops / (tc_ms * 1e-3) / 1e12
    tc_bytes = sum(KERNEL_TENSORS[k] for k in BWD_TC) * tensor_bytes
    tc_gbs = tc_bytes / (tc_ms * 1e-3) / 1e9
    # whole-step bounds: analytic FLOP against the tensor peak, compulsory bytes (every kernel's own tensors once)
    # against the HBM peak; the larger fraction names the binding bound
    step_bytes = sum(KERNEL_TENSORS[k] for k in kernel_ms) * tensor_bytes
    step_tensor_frac = (f_fwd + f_bwd) / (ms_step * 1e-3) / 1e12 / peak
    step_hbm_frac = step_bytes / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"]
    fwd_hbm_frac = KERNEL_TENSORS["fwd"] * tensor_bytes / (ms_fwd / args.steps * 1e-3) / 1e9 / peaks["hbm_gbs"]
    traffic = NCU_TRAFFIC_BYTES.get(args.workload)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "variant": args.variant, "B": wl.B, "H": wl.H, "N": wl.N, "d": wl.d, "per_gpu": True,
                   "timed_regions": len(regions),
                   "l2": "16 resident tensors of %.0f MB each, larger than the 126 MB L2; no flush" % (x["Q"].numel() * 2 / 1e6)},
        "fwd": dict({"tflops": fwd_tf, "ms": ms_fwd / args.steps, "cycles": cycles(ms_fwd / args.steps),
                     "frac": fwd_tf / peak, "hbm_frac": fwd_hbm_frac}, **fracs(fwd_tf)),
        "bwd": dict({"tflops": bwd_tf, "ms": ms_bwd / args.steps, "cycles": cycles(ms_bwd / args.steps),
                     "frac": bwd_tf / peak}, **fracs(bwd_tf)),
        "frac_of_burst_peak": value / world / peaks["bf16_tflops"],
        # the first timed region alone: the GPU has not reached its power cap yet (compare with the burst peak)
        "first_region": {"ms_per_step": regions[0] / args.steps,
                         "value": world * (f_fwd + f_bwd) / (regions[0] / args.steps * 1e-3) / 1e12,
                         "frac_of_burst_peak": (f_fwd + f_bwd) / (regions[0] / args.steps * 1e-3) / 1e12 / peaks["bf16_tflops"]},
        "kernels_ms": kernel_ms,
        "kernels_cycles": {k: cycles(v) for k, v in kernel_ms.items()},
        "kernels_share": {k: v / total_k for k, v in kernel_ms.items()},
        "kernels_executed_tflops": {k: KERNEL_GEMMS[k] * unit_flops / (v * 1e-3) / 1e12 for k, v in kernel_ms.items() if KERNEL_GEMMS[k]},
        "roofline": {"bound": "tensor" if step_tensor_frac >= step_hbm_frac else "hbm",
                     "kernel": "+".join(BWD_TC), "achieved": credited, "peak": peak, "unit": "TFLOP/s",
                     "frac": credited / peak, "peak_source": peak_note,
                     "achieved_executed": executed, "frac_executed": executed / peak,
                     "note": "achieved = the method's own %d GEMM units of the backward / summed duration of the three "
                             "tensor-core passes; achieved_executed counts the %d units they execute (scores recomputed per pass)"
                             % (credited_units, sum(KERNEL_GEMMS[k] for k in BWD_TC)),
                     "flops_per_launch": credited_units * unit_flops,
                     "flops_executed_per_launch": sum(KERNEL_GEMMS[k] for k in BWD_TC) * unit_flops,
                     "traffic": None if not traffic else sum(traffic[k] for k in BWD_TC),
                     "hbm": {"achieved": tc_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": tc_gbs / peaks["hbm_gbs"],
                             "bytes_per_launch": tc_bytes},
                     "step": {"tensor_frac": step_tensor_frac, "hbm_frac": step_hbm_frac, "bytes": step_bytes}},
        "e2e": None if ms_e2e is None else {
            "value": world * (f_fwd + f_bwd) / (ms_e2e * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_e2e,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "pipeline": "%d batch chunks; copy-in, compute and copy-out on three streams" % n_chunks},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if rms is not None:
        ms_nf, ms_nb = rms
        line["qk_rmsnorm"] = {
            "fwd_ms": ms_nf, "bwd_ms": ms_nb,
            "fwd_gbs": 8 * tensor_bytes / (ms_nf * 1e-3) / 1e9, "bwd_gbs": 12 * tensor_bytes / (ms_nb * 1e-3) / 1e9,
            "fwd_frac_of_hbm_peak": 8 * tensor_bytes / (ms_nf * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "bwd_frac_of_hbm_peak": 12 * tensor_bytes / (ms_nb * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "note": "forward reads 4 and writes 4 tensors, backward reads 8 and writes 4; time includes torch's output allocation"}
    if not args.no_cpu_baseline and world == 1:
        v, cores, desc, _, _ = oracle_sample(args.workload)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
