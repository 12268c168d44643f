"""Scaling sweep of the square NVFP4 Newton-Schulz step and of the quantiser.

    python -m paper_2607_04422_b200.sweep [--max-size 16384] [--reps 5]

Square Gaussian inputs (seed 1) from 512 to the maximum size in powers of two; 1 to 8
iterations for the step; prints one JSON line per case with the achieved algorithmic and
dense-equivalent TFLOP/s and, for fp4_quantize, the achieved GB/s."""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as fp4
from . import workloads


def _time(fn, reps, stream):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fn(); fn()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(reps):
        e0.record(stream); fn(); e1.record(stream)
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    return best


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--max-size", type=int, default=16384)
    ap.add_argument("--reps", type=int, default=5)
    a = ap.parse_args()
    stream = torch.cuda.current_stream()
    size = 512
    while size <= a.max_size:
        G = torch.from_numpy(workloads.sweep_square(size)).cuda()
        out = torch.empty_like(G)
        codes = torch.empty((size, size // 2), dtype=torch.uint8, device="cuda")
        scales = torch.empty(fp4.fp4_scale_bytes(size, size), dtype=torch.uint8, device="cuda")
        ts = torch.empty(1, device="cuda")
        ms = _time(lambda: fp4.fp4_quantize(G, codes, scales, ts, 0, stream), a.reps, stream)
        print(json.dumps({"case": "fp4_quantize", "size": size, "ms": round(ms, 4),
                          "gbs": round(size * size * 8.5625 / ms / 1e6, 1)}), flush=True)
        ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(size, size, 8), dtype=torch.uint8, device="cuda")
        for steps in range(1, 9):
            ms = _time(lambda: fp4.fp4_root_ns(G, out, steps, None, ws, stream), a.reps, stream)
            alg = steps * 4.0 * size ** 3
            print(json.dumps({"case": "fp4_root_ns", "size": size, "steps": steps, "ms": round(ms, 4),
                              "tflops_algorithmic": round(alg / ms / 1e9, 1),
                              "tflops_dense_equivalent": round(1.5 * alg / ms / 1e9, 1),
                              "pct_of_9pf": round(alg / ms / 1e9 / 90.0, 2)}), flush=True)
        status = fp4.fp4_last_device_status(ws)
        assert status == 0, status
        del G, out, ws, codes, scales
        size *= 2


if __name__ == "__main__":
    main()
