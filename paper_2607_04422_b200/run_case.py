"""Runs the Root Newton-Schulz step on one seeded synthetic matrix and prints its timing.

    python -m paper_2607_04422_b200.run_case --m 3072 --n 8192 --steps 5 --reps 3

A small, self-contained driver for profiling one shape (e.g. under ncu) or trying the
library from the command line.  Inputs come from workloads.gradient_like."""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as fp4
from . import workloads


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--m", type=int, default=3072)
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--quantize-only", action="store_true", help="time fp4_quantize instead of the NS step")
    ap.add_argument("--momentum", choices=["rtn", "sr"], help="time fp4_momentum_update instead of the NS step")
    ap.add_argument("--adamw", choices=["rtn", "sr"], help="time fp4_adamw_update on m*n BF16 parameters instead")
    a = ap.parse_args()
    if a.adamw:
        n = a.m * a.n
        gen = torch.Generator(device="cuda").manual_seed(a.seed)
        W = (torch.randn(n, generator=gen, device="cuda") * 0.05).to(torch.bfloat16)
        Gb = (torch.randn(n, generator=gen, device="cuda") * 1e-2).to(torch.bfloat16)
        mc, vc = (torch.zeros(n // 2, dtype=torch.uint8, device="cuda") for _ in range(2))
        ms, vs = (torch.zeros(n // 16, dtype=torch.int16, device="cuda") for _ in range(2))
        vm = torch.zeros(n // 256, dtype=torch.int16, device="cuda")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times = []
        for t in range(1, a.reps + 1):
            e0.record()
            fp4.fp4_adamw_update(W, Gb, mc, ms, vc, vs, vm, lr=1e-3, step=t,
                                 flags=fp4.FP4_MOM_FLAG_SR if a.adamw == "sr" else 0, seed=t)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        print(json.dumps({"case": "fp4_adamw_update", "mode": a.adamw, "params": n, "ms": times,
                          "gbs_best": n * 8.515625 / min(times) / 1e6}))
        return
    G = torch.from_numpy(workloads.gradient_like(a.m, a.n, seed=a.seed)).cuda()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    if a.momentum:
        codes = torch.zeros((a.m, a.n // 2), dtype=torch.uint8, device="cuda")
        scales = torch.zeros((a.m, a.n // 16), dtype=torch.int16, device="cuda")
        M = torch.empty_like(G)
        hist = torch.zeros(8192, dtype=torch.int32, device="cuda")
        flags = fp4.FP4_MOM_FLAG_SR if a.momentum == "sr" else 0
        for i in range(a.reps):
            e0.record(stream)
            fp4.fp4_momentum_update(G, codes, scales, M, hist, 0.95, 1.0, flags, i)
            e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        nbytes = a.m * a.n * 9.25
        print(json.dumps({"case": "fp4_momentum_update", "mode": a.momentum, "m": a.m, "n": a.n, "ms": times,
                          "gbs_best": nbytes / min(times) / 1e6}))
        return
    if a.quantize_only:
        codes = torch.empty((a.m, a.n // 2), dtype=torch.uint8, device="cuda")
        scales = torch.empty(fp4.fp4_scale_bytes(a.m, a.n), dtype=torch.uint8, device="cuda")
        ts = torch.empty(1, device="cuda")
        for _ in range(a.reps):
            e0.record(stream)
            fp4.fp4_quantize(G, codes, scales, ts)
            e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        nbytes = a.m * a.n * (4 + 4 + 0.5625)
        print(json.dumps({"case": "fp4_quantize", "m": a.m, "n": a.n, "ms": times,
                          "gbs_best": nbytes / min(times) / 1e6}))
        return
    out = torch.empty_like(G)
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(a.m, a.n, a.steps), dtype=torch.uint8, device="cuda")
    for _ in range(a.reps):
        e0.record(stream)
        fp4.fp4_root_ns(G, out, a.steps, None, ws)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    status = fp4.fp4_last_device_status(ws)
    s, l = min(a.m, a.n), max(a.m, a.n)
    alg = a.steps * (3.0 * s * s * l + s ** 3)
    print(json.dumps({"case": "fp4_root_ns", "m": a.m, "n": a.n, "steps": a.steps, "ms": times, "status": status,
                      "tflops_algorithmic_best": alg / min(times) / 1e9}))


if __name__ == "__main__":
    main()
