"""Run the forward call of one benchmark configuration a few times (for profilers and quick looks).

    python -m paper_2311_15806_b200.run_case cfg2 [--launches 3] [--kernel K] [--int8-copy]

Loads the seeded synthetic layer, expands the weights, quantizes the activations and launches the expanded GEMM
`--launches` times; prints the CUDA-event time of the last launch.  Nothing is checked here: parity lives in tests/.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from . import build as pipe_build
from . import synth
from .runner import LayerRunner


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("workload")
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--kernel", type=int, default=0, help="force a GEMM kernel (pipe_diag_select_kernel)")
    ap.add_argument("--int8-copy", action="store_true",
                    help="the layer also keeps its codes as int8 in the tensor-core operand layout (pipe_layer_desc.int8_copy)")
    args = ap.parse_args()
    pipe_build.build()
    B.lib()
    spec = synth.paper_workloads()[args.workload]
    run = LayerRunner(spec, int8_copy=args.int8_copy)
    run.load()
    run.expand()
    run.quantize()
    B.pipe_diag_select_kernel(args.kernel)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(max(1, args.launches)):
        e0.record()
        run.forward()
        e1.record()
    torch.cuda.synchronize()
    st = B.pipe_poll_status()
    print(f"{args.workload}: forward {e0.elapsed_time(e1) * 1e3:.1f} us (last of {args.launches} launches), status {B.pipe_status_string(st)}")
    if st != B.PIPE_OK:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
