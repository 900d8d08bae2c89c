#!/usr/bin/env python
"""Benchmark of the residual-expanded quantized layer (one pass of the whole hot path per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step = expand the fp32 weights + quantize the activations of every ensemble branch + the
(grouped) expanded GEMM, on one seeded synthetic batch.  With N > 1 (torchrun) every rank runs an
independent replica of the same workload on its own GPU (the path has no exchange step).
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
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

DEFAULT_WORKLOAD = "cfg2"
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
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("cfg2", "forward"): 27.573504e6 + 49.119488e6,      # profiles/ncu_tc_forward_kernel_cfg2.txt
    ("cfg4a_t16", "forward"): 56.678656e6 + 0.802048e6,  # profiles/ncu_stream_forward_kernel_cfg4a_t16.txt
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


def time_oracle_sample(spec, target_seconds: float = 12.0):
    """The CPU oracle, as it stands, on a bounded sample of the workload: full weight expansion,
    then activation quantization + forward of every branch on the first `n` token rows."""
    from oracle import pipe_oracle as O
    from paper_2311_15806_b200 import synth
    O.build()
    cores = O.threads()
    W = synth.make_weights(spec)
    G = spec.O // spec.g
    n_keep = O.keep_groups(G, spec.gamma)
    t0 = time.perf_counter()
    e = O.expand(W, spec.bits, spec.K, spec.g, n_keep)
    t_expand = time.perf_counter() - t0
    split = O.balanced_split(spec.K, spec.M)

    def rows_of(n, m):
        if spec.conv is not None:
            x4 = synth.make_conv_input(spec, m)
            return synth.im2col_rows(x4, spec.conv, np.arange(n))
        return synth.make_activations(spec.with_tokens(max(n, 1)), m)[:n]

    def run(n):
        xs = [rows_of(n, m) for m in range(spec.M)]
        t1 = time.perf_counter()
        k0 = 0
        for m in range(spec.M):
            xq, sx = O.quantize_act(xs[m])
            O.forward(e, xq, sx, k0, k0 + int(split[m]))
            k0 += int(split[m])
        return time.perf_counter() - t1

    n = min(spec.T, 8)
    t_small = max(run(n), 1e-4)
    n_big = int(min(spec.T, max(n, n * target_seconds / t_small)))
    t_big = run(n_big) if n_big > n else t_small
    per_token = t_big / n_big
    est_step = t_expand + per_token * spec.T
    return {"value": spec.T / est_step, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": (f"full weight expansion ({t_expand:.2f} s) + quantize and forward of all {spec.M} branch(es) "
                       f"on the first {n_big} of {spec.T} token rows ({t_big:.2f} s), extrapolated to the whole step"),
            "seconds_per_step_estimate": est_step}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = workload_spec(args.workload)
    vals = []
    base = None
    budget = max(3.0, min(12.0, 60.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        base = time_oracle_sample(spec, target_seconds=budget)
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
        B.pipe_select_kernel(args.kernel)

    spec = workload_spec(args.workload)
    peaks = load_peaks()
    run = LayerRunner(spec)
    run.load()
    T = run.T
    in_bytes = sum(x.numel() * 4 for x in run.x) + run.W.numel() * 4
    flush = None
    if in_bytes <= 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
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
        run.expand()
        ev[i][1].record()
        run.quantize()
        ev[i][2].record()
        run.forward()
        ev[i][3].record()
    sync_all()
    wall = time.perf_counter() - wall0
    launches = B.pipe_launch_count() - launches0
    t_expand = [ev[i][0].elapsed_time(ev[i][1]) for i in range(args.steps)]
    t_quant = [ev[i][1].elapsed_time(ev[i][2]) for i in range(args.steps)]
    t_fwd = [ev[i][2].elapsed_time(ev[i][3]) for i in range(args.steps)]
    total_ms = sum(ev[i][0].elapsed_time(ev[i][3]) for i in range(args.steps))
    total_ms = max_over_ranks(total_ms, world, "cuda")
    ms_per_step = total_ms / args.steps
    tokens_per_s = whole_job_tokens_per_s(world, T, args.steps, total_ms)
    macs = run.macs_per_token() * T

    # ---- the GEMM kernel alone: back-to-back launches (one CUDA graph when capture works, so that
    # the host does not pace ~10 us kernels), rotating over copies of the blob whose total size
    # exceeds L2 so that weights are streamed from HBM every launch
    reps = 20
    blobs = run.blob_copies(0 if flush is None else 2 * L2_BYTES)
    blobs = blobs[:reps]
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
    # The clock sampler (one nvidia-smi sample per 100 ms) keeps running through this loop, which therefore
    # goes on for at least half a second: the timed steps above are over within a few milliseconds.
    launch_ms = []
    t_loop = time.perf_counter()
    while len(launch_ms) < 5 or (time.perf_counter() - t_loop < 0.6 and len(launch_ms) < 20000):
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        k0.record()
        if graph is not None:
            graph.replay()
        else:
            launch_all()
        k1.record()
        torch.cuda.synchronize()
        launch_ms.append(k0.elapsed_time(k1) / reps)
    fwd_launch_ms = statistics.median(launch_ms)
    clocks = sampler.stop()
    del blobs
    st = B.pipe_poll_status()
    if st != B.PIPE_OK:
        raise SystemExit(f"device status after the kernel timing loop: {B.pipe_status_string(st)}")

    # ---- end to end: host buffers in, host buffer out, copies inside the timed region ------------
    hW = run.W.cpu().pin_memory()
    hx = [x.cpu().pin_memory() for x in run.x]
    hy = [torch.empty(y.shape, dtype=y.dtype).pin_memory() for y in run.y]
    e2e_steps = max(1, min(args.steps, 3))
    for it in range(1 + e2e_steps):
        if it == 1:
            sync_all()
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
        run.W.copy_(hW, non_blocking=True)
        for m in range(len(hx)):
            run.x[m].copy_(hx[m], non_blocking=True)
        run.step()
        for m in range(len(hy)):
            hy[m].copy_(run.y[m], non_blocking=True)
    e1.record()
    sync_all()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, world, "cuda")
    h2d = hW.numel() * 4 + sum(x.numel() * 4 for x in hx)
    d2h = sum(y.numel() * 4 for y in hy)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel -----------------------------------------------------------
    phases = {"expand": statistics.mean(t_expand), "quantize": statistics.mean(t_quant), "forward": statistics.mean(t_fwd)}
    dominant = max(phases, key=phases.get)
    int8_peak_burst = 2.0 * peaks["bf16_tflops"]
    int8_peak_sust = 2.0 * peaks["bf16_tflops_sustained"]
    fwd_s = fwd_launch_ms * 1e-3   # per-launch duration of the GEMM kernel, back-to-back launches
    fwd_tops = 2.0 * macs / fwd_s / 1e12
    fwd_gbs = run.forward_bytes() / fwd_s / 1e9
    ai = 2.0 * macs / run.forward_bytes()
    ridge = int8_peak_sust * 1e12 / (peaks["hbm_gbs"] * 1e9)
    if dominant == "forward":
        if ai >= ridge:
            roof = {"kernel": "expanded GEMM (pipe_expanded_linear / pipe_ensemble_forward)", "bound": "tensor",
                    "achieved": fwd_tops, "peak": int8_peak_sust, "unit": "TOP/s",
                    "frac": fwd_tops / int8_peak_sust,
                    "peak_note": f"2 x bf16 sustained of {peaks['source']} (int8:bf16 nominal ratio 4.5:2.25)"}
        else:
            roof = {"kernel": "expanded GEMM (pipe_expanded_linear / pipe_ensemble_forward)", "bound": "hbm",
                    "achieved": fwd_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": fwd_gbs / peaks["hbm_gbs"],
                    "peak_note": f"copy bandwidth of {peaks['source']}"}
    else:
        nbytes = run.expand_bytes() if dominant == "expand" else run.quantize_bytes()
        gbs = nbytes / (phases[dominant] * 1e-3) / 1e9
        roof = {"kernel": f"{dominant} kernels", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "peak_note": f"copy bandwidth of {peaks['source']}"}
    # DRAM read + write bytes per launch of the dominant kernel from one ncu capture of this same
    # command line (summaries under profiles/); None where no capture of the current kernel exists.
    roof["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get((spec.name, dominant))

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle_sample(spec)

    line = {"metric": "expanded_layer_tokens_per_s", "value": tokens_per_s, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": dict(config_of(spec), l2="flush_between_steps" if flush is not None else "inputs_exceed_l2",
                           distinct_branch_inputs=run.distinct_inputs, multi_gpu="independent replicas"),
            "effective_tops_whole_step": 2.0 * macs * world / (ms_per_step * 1e-3) / 1e12,
            "forward": {"ms": fwd_launch_ms, "timing": ("cuda graph of 20 launches" if graph is not None else "20 back-to-back launches")
                        + (", blob copies rotated (> 2 x L2)" if flush is not None else ""),
                        "ms_in_step": phases["forward"], "effective_tops": fwd_tops, "gbs": fwd_gbs,
                        "frac_int8_peak_sustained": fwd_tops / int8_peak_sust, "frac_int8_peak_burst": fwd_tops / int8_peak_burst,
                        "frac_int8_nominal_4500": fwd_tops / 4500.0, "frac_hbm": fwd_gbs / peaks["hbm_gbs"],
                        "arithmetic_intensity": ai},
            "phases_ms": phases, "roofline": roof, "clocks": clocks,
            "e2e": {"value": world * T / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": int(launches), "wall_s_timed_region": wall, "cpu_baseline": cpu}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--kernel", type=int, default=None, help="force a GEMM kernel (see pipe_select_kernel)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args(argv)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
