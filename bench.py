#!/usr/bin/env python
"""Benchmark of the residual-expanded quantized layer (one pass of the whole hot path per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step runs the whole hot path on one seeded synthetic batch -- expand the fp32 weights, quantize the
activations of every ensemble branch, run the (grouped) expanded GEMM -- with every phase timed on its own.
The paper expands a network once, offline (Sec. 4.1), so `value` is the ONLINE path (quantize + GEMM) and the
expansion is reported beside it as its own phase.  The headline workload is the largest configuration
(cfg5); with one GPU the line also carries a `workloads` table with the GEMM of every configuration, timed
alone, against the integer tensor peak measured in the same run (large token counts) or the measured copy
bandwidth (T <= 16).  With N > 1 (torchrun) every rank runs an independent replica of the headline workload on
its own GPU (the path has no exchange step).  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

DEFAULT_WORKLOAD = "cfg5"
TABLE_WORKLOADS = (["cfg1", "cfg2", "cfg3a", "cfg3b"] + [f"cfg4{ab}_t{T}" for ab in "ab" for T in (1, 16, 128, 1024, 4096)]
                   + ["cfg5"])
# rows measured once more on a layer that keeps its codes as int8 in the tensor-core operand layout as well
# (pipe_layer_desc.int8_copy: twice the packed bytes of 4-bit codes in HBM, no widening in shared memory)
INT8_COPY_WORKLOADS = ["cfg3a", "cfg3b", "cfg4a_t128", "cfg4a_t1024", "cfg4a_t4096", "cfg4b_t4096"]
L2_BYTES = 126 * 1024 * 1024


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def workload_spec(name: str):
    from paper_2311_15806_b200 import synth
    w = synth.paper_workloads()
    if name not in w:
        raise SystemExit(f"unknown workload {name!r}; choose from {sorted(w)}")
    return w[name]


# ------------------------------------------------------------------------------------------------
# DRAM read + write bytes of ONE launch of the GEMM kernel, from one ncu capture per workload of this same
# program (summaries under profiles/, named in the comment).  A workload without a capture of the present
# kernel has no entry and reports null.
NCU_DRAM_BYTES_PER_LAUNCH = {
    "cfg2": 29317632 + 51065600,           # profiles/ncu_tc2_forward_kernel_cfg2.txt
    "cfg3a": 9438976 + 49971456,           # profiles/ncu_tc2_forward_kernel_cfg3a.txt
    "cfg4a_t4096": 91033600 + 313256192,   # profiles/ncu_tc2_forward_kernel_cfg4a_t4096.txt
    "cfg5": 478397440 + 1029014784,        # profiles/ncu_tc2_forward_kernel_cfg5.txt
    "cfg4a_t1": 56559616 + 98304,          # profiles/ncu_stream_forward_kernel_cfg4a_t1.txt
    "cfg4a_t16": 56688128 + 303872,         # profiles/ncu_stream_forward_kernel_cfg4a_t16.txt
    "cfg4a_t4096+int8_copy": 149131520 + 316639744,   # profiles/ncu_tc2_forward_kernel_cfg4a_t4096_int8_copy.txt
    "cfg3b+int8_copy": 31190784 + 930048,           # profiles/ncu_tc2_forward_kernel_cfg3b_int8_copy.txt
}


def max_over_ranks(value_ms: float, world: int, device) -> float:
    """Replicas run independently; the job's time is that of its slowest rank."""
    if world <= 1:
        return float(value_ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, tokens_per_replica: int, steps: int, total_ms: float) -> float:
    """Aggregate over all replicas: every rank processes its own `tokens_per_replica` per step."""
    return world * tokens_per_replica * steps / (total_ms * 1e-3)


class OracleTimer:
    """The CPU oracle, as it stands, on a bounded sample of a workload: the weights are expanded once (as the
    paper does, offline), then activation quantization + forward of every branch run on the first n token rows."""

    def __init__(self, spec):
        from oracle import pipe_oracle as O
        from paper_2311_15806_b200 import synth
        O.build()
        self.O, self.synth, self.spec = O, synth, spec
        self.cores = O.threads()
        W = synth.make_weights(spec)
        n_keep = O.keep_groups(spec.O // spec.g, spec.gamma)
        t0 = time.perf_counter()
        self.e = O.expand(W, spec.bits, spec.K, spec.g, n_keep)
        self.t_expand = time.perf_counter() - t0
        self.split = O.balanced_split(spec.K, spec.M)

    def _rows(self, n, m):
        spec = self.spec
        if spec.conv is not None:
            return self.synth.im2col_rows(self.synth.make_conv_input(spec, m), spec.conv, np.arange(n))
        return self.synth.make_activations(spec.with_tokens(max(n, 1)), m)[:n]

    def run(self, n: int) -> float:
        xs = [self._rows(n, m) for m in range(self.spec.M)]
        t1 = time.perf_counter()
        k0 = 0
        for m in range(self.spec.M):
            xq, sx = self.O.quantize_act(xs[m])
            self.O.forward(self.e, xq, sx, k0, k0 + int(self.split[m]))
            k0 += int(self.split[m])
        return time.perf_counter() - t1

    def sample(self, target_seconds: float) -> dict:
        spec = self.spec
        n = min(spec.T, 8)
        t_small = max(self.run(n), 1e-4)
        n_big = int(min(spec.T, max(n, n * target_seconds / t_small)))
        t_big = self.run(n_big) if n_big > n else t_small
        est_step = t_big / n_big * spec.T
        return {"value": spec.T / est_step, "unit": "tokens/s", "cores": self.cores, "kind": "oracle",
                "sample": (f"weights expanded once beforehand ({self.t_expand:.2f} s, not in the value); quantize and forward "
                           f"of all {spec.M} branch(es) on the first {n_big} of {spec.T} token rows ({t_big:.2f} s), "
                           f"extrapolated to the whole step"),
                "seconds_per_step_estimate": est_step, "expand_seconds": self.t_expand}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = workload_spec(args.workload)
    timer = OracleTimer(spec)
    vals = []
    base = None
    budget = max(2.0, min(12.0, 60.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        base = timer.sample(budget)
        if i >= args.warmup:
            vals.append(base["value"])
    v = statistics.mean(vals)
    line = {"impl": "reference", "metric": "expanded_layer_tokens_per_s", "value": v, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * spec.T / v,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": config_of(spec), "cpu_baseline": dict(base, value=v),
            "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def config_of(spec):
    return {"workload": spec.name, "out_features": spec.O, "in_features": spec.I, "tokens": spec.T,
            "weight_bits": spec.bits, "act_bits": 8, "orders": spec.K, "group_size": spec.g, "gamma": spec.gamma,
            "branches": spec.M, "seed": spec.seed, "conv": list(spec.conv) if spec.conv else None}


# ------------------------------------------------------------------------------------------------
def measure_int8_peak(B, torch, device_index):
    """The integer tensor peak of THIS device, in this run: the library's issue-bound probe (tcgen05.mma kind::i8,
    M = 128, N = 256, operands resident in shared memory) as a burst and over a seconds-long loop, and
    torch._int_mm on 8192^3 as an independent cross-check."""
    def timed(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3, out

    B.pipe_diag_mma_i8_rate(256, 2000)
    torch.cuda.synchronize()
    burst = 0.0
    for _ in range(5):
        dt, ops = timed(lambda: B.pipe_diag_mma_i8_rate(256, 40000))   # about 3 ms
        burst = max(burst, ops / dt / 1e12)
    sampler = ClockSampler(device_index)
    sampler.start()
    t0 = time.perf_counter()
    sus = []
    while time.perf_counter() - t0 < 1.5:
        dt, ops = timed(lambda: B.pipe_diag_mma_i8_rate(256, 1000000))  # about 70 ms
        sus.append(ops / dt / 1e12)
    clocks = sampler.stop()
    out = {"probe_burst": burst, "probe_sustained": statistics.median(sus[len(sus) // 2:]) if sus else None,
           "probe": "tcgen05.mma.kind::i8 M128 N256 K32, one CTA per SM, operands resident in shared memory",
           "sustained_clocks": clocks, "unit": "TOP/s", "nominal": 4500.0}
    try:
        a = torch.randint(-127, 128, (8192, 8192), dtype=torch.int8, device="cuda")
        b = torch.randint(-127, 128, (8192, 8192), dtype=torch.int8, device="cuda")
        for _ in range(3):
            torch._int_mm(a, b)
        best = 0.0
        for _ in range(10):
            dt, _ = timed(lambda: torch._int_mm(a, b))
            best = max(best, 2.0 * 8192.0 ** 3 / dt / 1e12)
        out["int_mm_8192"] = best
        del a, b
    except Exception as exc:   # the cross-check is a library call outside this repository
        out["int_mm_8192"] = None
        out["int_mm_note"] = f"{type(exc).__name__}: {exc}"[:120]
    if B.pipe_poll_status() != B.PIPE_OK:
        raise SystemExit("device status after the tensor-peak probe is not ok")
    return out


def time_forward_alone(run, torch, device_index, flush_needed: bool, min_seconds: float = 0.4):
    """The GEMM call alone: graphs of 20 back-to-back launches (so that the host does not pace kernels of a few
    microseconds), rotating over copies of the blob whose total size exceeds L2 when the weights alone would fit
    it, repeated for `min_seconds` while nvidia-smi samples the clocks.  Returns (median ms per launch, how, clocks)."""
    reps = 20
    blobs = run.blob_copies(2 * L2_BYTES if flush_needed else 0)[:reps]

    def launch_all():
        for r in range(reps):
            run.forward(blob=blobs[r % len(blobs)])
    for _ in range(2):
        launch_all()
    torch.cuda.synchronize()
    graph = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                launch_all()
        torch.cuda.current_stream().wait_stream(side)
        graph = g
    except Exception:
        graph = None
        torch.cuda.synchronize()
    sampler = ClockSampler(device_index)
    sampler.start()
    launch_ms = []
    t_loop = time.perf_counter()
    while len(launch_ms) < 5 or (time.perf_counter() - t_loop < min_seconds and len(launch_ms) < 20000):
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        k0.record()
        if graph is not None:
            graph.replay()
        else:
            launch_all()
        k1.record()
        torch.cuda.synchronize()
        launch_ms.append(k0.elapsed_time(k1) / reps)
    clocks = sampler.stop()
    how = ("cuda graph of 20 launches" if graph is not None else "20 back-to-back launches") + \
          (f", {len(blobs)} blob copies rotated (> 2 x L2)" if flush_needed else ", inputs exceed L2")
    del graph
    return statistics.median(launch_ms), min(launch_ms), how, clocks


def forward_row(run, spec, fwd_ms, fwd_best_ms, how, clocks, peaks, int8, sms: int = 148):
    """One row of the workloads table: the GEMM of one configuration against its roofline."""
    macs = run.macs_per_token() * run.T
    ops = 2.0 * macs
    nbytes = run.forward_bytes()
    tops = ops / (fwd_ms * 1e-3) / 1e12
    gbs = nbytes / (fwd_ms * 1e-3) / 1e9
    ai = ops / nbytes
    ridge = int8["probe_burst"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    bound = "tensor" if ai >= ridge else "hbm"
    row = {"workload": spec.name, "tokens": run.T, "forward_ms": fwd_ms, "forward_ms_best": fwd_best_ms, "timing": how,
           "ops_per_launch": ops, "bytes_per_launch": nbytes, "effective_tops": tops, "gbs": gbs,
           "arithmetic_intensity": ai, "bound": bound,
           "frac_int8_probe_burst": tops / int8["probe_burst"],
           # (the timing loop runs for a few tenths of a second: long enough for a dense kernel to meet the power cap
           # that the 1.5 s probe loop settles under, so that figure is given beside the burst one)
           "frac_int8_probe_sustained": (tops / int8["probe_sustained"]) if int8.get("probe_sustained") else None,
           "frac_int8_int_mm": (tops / int8["int_mm_8192"]) if int8.get("int_mm_8192") else None,
           "frac_int8_2x_bf16_burst": tops / (2.0 * peaks["bf16_tflops"]),
           "frac_int8_nominal_4500": tops / 4500.0,
           # per clock and SM against the tensor pipe's issue rate (8192 MAC), at the SM clock sampled during this loop:
           # a seconds-long loop of a dense kernel runs into the power cap, so its clock is below the probe's burst clock
           "mac_per_clk_per_sm": (macs / (fwd_ms * 1e-3) / (clocks["sm_mhz"] * 1e6) / sms) if clocks.get("sm_mhz") else None,
           "frac_issue_rate_at_sampled_clock": (macs / (fwd_ms * 1e-3) / (clocks["sm_mhz"] * 1e6) / sms / 8192.0) if clocks.get("sm_mhz") else None,
           "frac_hbm_copy": gbs / peaks["hbm_gbs"], "frac_hbm_nominal_8000": gbs / 8000.0,
           "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(spec.name),
           "clocks": clocks}
    return row


def roofline_of(row, peaks, int8):
    """The `roofline` object for the GEMM of one workload (always the expanded GEMM, never another phase)."""
    kernel = "expanded GEMM (pipe_expanded_linear / pipe_ensemble_forward / pipe_expanded_conv2d)"
    if row["bound"] == "tensor":
        return {"kernel": kernel, "bound": "tensor", "achieved": row["effective_tops"], "peak": int8["probe_burst"],
                "unit": "TOP/s", "frac": row["frac_int8_probe_burst"],
                "peak_note": "issue-bound tcgen05.mma kind::i8 probe of this run, burst (the kernel is timed alone); "
                             f"torch._int_mm 8192^3 gave {int8.get('int_mm_8192')} and 2 x bf16 burst of {peaks['source']} "
                             f"is {2.0 * peaks['bf16_tflops']}",
                "traffic": row["traffic"]}
    return {"kernel": kernel, "bound": "hbm", "achieved": row["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": row["frac_hbm_copy"], "peak_note": f"copy bandwidth of {peaks['source']}", "traffic": row["traffic"]}


def host_time_per_forward_call(run, B, torch, calls: int = 300):
    """Host microseconds a forward call takes on repeat calls, outside any graph (arguments marshalled once)."""
    import ctypes as C
    lib = B.lib()
    M = run.M
    n = len(run.xq)
    PA = C.c_void_p * M
    xp = PA(*[int(run.xq[m if n > 1 else 0].data_ptr()) for m in range(M)])
    sp = PA(*[int(run.sx[m if n > 1 else 0].data_ptr()) for m in range(M)])
    yp = PA(*[int(run.y[m].data_ptr()) for m in range(M)])
    stream = int(torch.cuda.current_stream().cuda_stream)
    desc = C.byref(run.desc)
    blob = int(run.blob.data_ptr())
    T, ldx, ldy = run.T, run.spec.I, run.spec.O

    def call():
        return lib.pipe_ensemble_forward(desc, blob, xp, T, ldx, sp, None, yp, ldy, 0, None, stream)
    for _ in range(20):
        if call() != B.PIPE_OK:
            return None
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(calls):
        call()
    dt = time.perf_counter() - t0
    torch.cuda.synchronize()
    return dt / calls * 1e6


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2311_15806_b200 import binding as B
    from paper_2311_15806_b200 import build as pipe_build
    from paper_2311_15806_b200.runner import LayerRunner

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        pipe_build.build()
    if world > 1:
        dist.barrier()
    B.lib()
    if args.kernel is not None:
        B.pipe_diag_select_kernel(args.kernel)
    nvtx = torch.cuda.nvtx

    spec = workload_spec(args.workload)
    peaks = load_peaks()
    warmup = max(args.warmup, 3)
    run = LayerRunner(spec)
    W_host = run.host_weights()
    x_host = run.host_inputs()
    sha = None
    if rank == 0:
        sha = {"W": hashlib.sha256(W_host.tobytes()).hexdigest()}
        for m, x in enumerate(x_host):
            if x is not None:
                sha[f"x{m}"] = hashlib.sha256(x.tobytes()).hexdigest()
    run.load(W_host, x_host)
    del W_host, x_host
    T = run.T
    online_in_bytes = sum(x.numel() * 4 for x in run.x)
    flush = None
    if online_in_bytes + run.layout.blob_bytes <= 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(warmup):
        run.step()
    sync_all()
    st = B.pipe_poll_status()
    if st != B.PIPE_OK:
        raise SystemExit(f"device status after warm-up: {B.pipe_status_string(st)}")

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    launches0 = B.pipe_launch_count()
    sampler = ClockSampler(local)
    sampler.start()
    sync_all()
    wall0 = time.perf_counter()
    for i in range(args.steps):
        if flush is not None:
            flush.fill_(i & 0xff)
        ev[i][0].record()
        nvtx.range_push("pipe_expand_weights")
        run.expand()
        nvtx.range_pop()
        ev[i][1].record()
        nvtx.range_push("pipe_quantize_act")
        run.quantize()
        nvtx.range_pop()
        ev[i][2].record()
        nvtx.range_push("pipe_forward")
        run.forward()
        nvtx.range_pop()
        ev[i][3].record()
    sync_all()
    wall = time.perf_counter() - wall0
    step_clocks = sampler.stop()
    launches = B.pipe_launch_count() - launches0
    t_expand = [ev[i][0].elapsed_time(ev[i][1]) for i in range(args.steps)]
    t_quant = [ev[i][1].elapsed_time(ev[i][2]) for i in range(args.steps)]
    t_fwd = [ev[i][2].elapsed_time(ev[i][3]) for i in range(args.steps)]
    online_ms = max_over_ranks(sum(t_quant) + sum(t_fwd), world, "cuda")
    whole_ms = max_over_ranks(sum(ev[i][0].elapsed_time(ev[i][3]) for i in range(args.steps)), world, "cuda")
    ms_per_step = online_ms / args.steps
    tokens_per_s = whole_job_tokens_per_s(world, T, args.steps, online_ms)
    macs = run.macs_per_token() * T

    # ---- end to end: host buffers in, host buffer out, copies inside the timed region (the online path: the
    # activations travel every step; the expanded weights stay on the device as they do in deployment)
    hx = [x.cpu().pin_memory() for x in run.x]
    hy = [torch.empty(y.shape, dtype=y.dtype).pin_memory() for y in run.y]
    # The steps are pipelined the way a serving loop would: inputs go up on one stream, results come down on another,
    # device buffers are double, so step i's download overlaps step i + 1's upload (the link is full duplex) and both
    # overlap the kernels; every step's copies lie inside the timed region, which ends when the last result is on the host.
    e2e_steps = max(1, min(args.steps, 10))
    main_stream = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    xbuf = [run.x, [torch.empty_like(x) for x in run.x]]
    ybuf = [run.y, [torch.empty_like(y) for y in run.y]]
    ev_in, ev_cmp, ev_out = [None, None], [None, None], [None, None]
    for it in range(2 + e2e_steps):
        b = it & 1
        if it == 2:
            sync_all()
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
        with torch.cuda.stream(s_in):
            if it >= 2:
                s_in.wait_event(ev_cmp[b] if it > 2 else e0)   # the kernels of step it - 2 have read this input buffer
            for m in range(len(hx)):
                xbuf[b][m].copy_(hx[m], non_blocking=True)
            ev_in[b] = torch.cuda.Event()
            ev_in[b].record(s_in)
        main_stream.wait_event(ev_in[b])
        if ev_out[b] is not None:
            main_stream.wait_event(ev_out[b])                  # the download of step it - 2 has read this output buffer
        run.x, run.y = xbuf[b], ybuf[b]
        run.quantize()
        run.forward()
        ev_cmp[b] = torch.cuda.Event()
        ev_cmp[b].record(main_stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[b])
            for m in range(len(hy)):
                hy[m].copy_(ybuf[b][m], non_blocking=True)
            ev_out[b] = torch.cuda.Event()
            ev_out[b].record(s_out)
    for b in (0, 1):
        main_stream.wait_event(ev_out[b])
    e1.record()
    sync_all()
    run.x, run.y = xbuf[0], ybuf[0]
    del xbuf, ybuf
    e2e_ms = max_over_ranks(e0.elapsed_time(e1) / e2e_steps, world, "cuda")
    h2d = sum(x.numel() * 4 for x in hx)
    d2h = sum(y.numel() * 4 for y in hy)
    del hx, hy

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- the integer tensor peak of this device, then the GEMM of the headline workload alone -----------------
    int8 = measure_int8_peak(B, torch, local)
    fwd_ms, fwd_best, how, fclocks = time_forward_alone(run, torch, local, flush is not None)
    st = B.pipe_poll_status()
    if st != B.PIPE_OK:
        raise SystemExit(f"device status after the kernel timing loop: {B.pipe_status_string(st)}")
    sms = torch.cuda.get_device_properties(local).multi_processor_count
    head_row = forward_row(run, spec, fwd_ms, fwd_best, how, fclocks, peaks, int8, sms)
    phases = {"expand": statistics.mean(t_expand), "quantize": statistics.mean(t_quant), "forward": statistics.mean(t_fwd)}
    expand_gbs = run.expand_bytes() / (phases["expand"] * 1e-3) / 1e9
    quant_gbs = run.quantize_bytes() / (phases["quantize"] * 1e-3) / 1e9 if phases["quantize"] > 0 else None

    # ---- every configuration's GEMM (one GPU only: the other ranks of a multi-GPU run would idle meanwhile) -------
    table = []
    host_us = None
    if world == 1 and not args.no_table:
        for name, int8_copy in [(n, False) for n in TABLE_WORKLOADS] + [(n, True) for n in INT8_COPY_WORKLOADS]:
            if name == spec.name and not int8_copy:
                table.append(head_row)
                continue
            del run
            torch.cuda.empty_cache()
            s2 = workload_spec(name)
            run = LayerRunner(s2, int8_copy=int8_copy)
            run.load()
            run.expand()
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            run.quantize()
            torch.cuda.synchronize()
            q0.record()
            run.quantize()
            q1.record()
            torch.cuda.synchronize()
            small = sum(x.numel() * 4 for x in run.x) + run.layout.blob_bytes <= 2 * L2_BYTES
            try:
                ms, best, how2, ck = time_forward_alone(run, torch, local, small, min_seconds=0.3)
            except B.PipeError as exc:   # only with --kernel: the forced back end does not take this shape
                table.append({"workload": name, "tokens": run.T, "error": str(exc)})
                continue
            row = forward_row(run, s2, ms, best, how2, ck, peaks, int8, sms)
            row["quantize_ms"] = q0.elapsed_time(q1)
            if int8_copy:
                row["workload"] = name + "+int8_copy"
                row["weights"] = "int8 copy in the operand layout beside the packed codes"
                row["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get(row["workload"])
            if name == "cfg4a_t1" and not int8_copy:
                host_us = host_time_per_forward_call(run, B, torch)
                row["host_us_per_call"] = host_us
            st = B.pipe_poll_status()
            if st != B.PIPE_OK:
                raise SystemExit(f"device status after {name}: {B.pipe_status_string(st)}")
            table.append(row)
    del run
    torch.cuda.empty_cache()

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = OracleTimer(spec).sample(12.0)

    line = {"metric": "expanded_layer_tokens_per_s", "value": tokens_per_s, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": dict(config_of(spec), l2="flush_between_steps" if flush is not None else "inputs_exceed_l2",
                           distinct_branch_inputs=True if spec.M > 1 else False, multi_gpu="independent replicas",
                           step="online path: pipe_quantize_act of every branch input + the grouped expanded GEMM; the "
                                "one-off weight expansion (Sec. 4.1) runs every step too but is timed as its own phase"),
            "effective_tops_online_step": 2.0 * macs * world / (ms_per_step * 1e-3) / 1e12,
            "whole_path_ms_per_step": whole_ms / args.steps,
            "phases_ms": phases,
            "expand": {"ms": phases["expand"], "gbs": expand_gbs, "frac_hbm_copy": expand_gbs / peaks["hbm_gbs"],
                       "bytes": run_expand_bytes_note()},
            "quantize": {"ms": phases["quantize"], "gbs": quant_gbs,
                         "frac_hbm_copy": (quant_gbs / peaks["hbm_gbs"]) if quant_gbs else None},
            "forward": head_row, "roofline": roofline_of(head_row, peaks, int8), "int8_peak": int8,
            "hbm_peak": {"copy_gbs": peaks["hbm_gbs"], "source": peaks["source"], "nominal_gbs": 8000.0},
            "workloads": table, "clocks": dict(fclocks, during="the GEMM timing loop of the headline workload",
                                               steps=step_clocks),
            "e2e": {"value": world * T / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "pipeline": "double-buffered device inputs and outputs, upload and download on their own streams"},
            "gpu_launches": int(launches), "wall_s_timed_region": wall, "host_us_per_forward_call_cfg4a_t1": host_us,
            "sha256": sha, "cpu_baseline": cpu}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_expand_bytes_note() -> str:
    return ("per order: fp32 rows read (+ written as residual unless last) + both code layouts written; order 1 reads "
            "the weights once more for the row maximum")


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--kernel", type=int, default=None, help="force a GEMM kernel (see pipe_diag_select_kernel)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-table", action="store_true", help="skip the per-configuration GEMM table")
    return ap.parse_args(argv)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
