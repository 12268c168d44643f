"""Scaling sweep of the square NVFP4 Newton-Schulz step and of the quantiser.

    python -m paper_2607_04422_b200.sweep [--max-size 16384] [--reps 5]

Square Gaussian inputs (seed 1) from 512 to the maximum size in powers of two; 1 to 8
iterations for the step; prints one JSON line per case with the achieved algorithmic and
dense-equivalent TFLOP/s and, for fp4_quantize, the achieved GB/s.

    python -m paper_2607_04422_b200.sweep --stacks

times, instead, one batched call over four decoder blocks of the paper's timing shapes
(Section 4.3: d = 4096 / 6144, d_ff = 11008 / 13824, grouped-query attention with 8 KV
heads), separate and fused projections, next to the same Newton-Schulz iterations in BF16
on cuBLAS (torch.matmul, dense, clip and normalisation outside the timed region)."""
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


def _bf16_ns_ms(shapes, abcs, steps, stream):
    """The NS iterations of every matrix in BF16 with torch.matmul; inputs are unit-norm Gaussians."""
    xs = []
    for m, n in shapes:
        x = torch.randn((min(m, n), max(m, n)), device="cuda")
        xs.append((x / x.norm()).to(torch.bfloat16))

    def run():
        for x, (a, b, c) in zip(xs, abcs):
            for _ in range(steps):
                A = x @ x.T
                B = b * A + c * (A @ A)
                x = a * x + B @ x
    return _time(run, 3, stream)


def stacks(reps, stream):
    steps = 5
    for d, d_ff in ((4096, 11008), (6144, 13824)):
        for fused in (False, True):
            shapes = [(m, n) for _, m, n in workloads.gqa_stack_shapes(d, d_ff, fused=fused)]
            gen = torch.Generator(device="cuda"); gen.manual_seed(d + int(fused))
            Gs = [torch.randn((m, n), device="cuda", generator=gen) for m, n in shapes]
            outs = [torch.empty_like(g) for g in Gs]
            ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, steps), dtype=torch.uint8, device="cuda")
            ms = _time(lambda: fp4.fp4_root_ns_batched(Gs, outs, steps, None, ws, stream), reps, stream)
            assert fp4.fp4_last_device_status(ws) == 0
            alg = sum(steps * (3.0 * min(m, n) ** 2 * max(m, n) + min(m, n) ** 3) for m, n in shapes)
            del ws, outs
            abcs = [fp4.fp4_root_coeffs(m, n, steps) for m, n in shapes]
            bf16 = _bf16_ns_ms(shapes, abcs, steps, stream)
            print(json.dumps({"case": "stack", "d": d, "d_ff": d_ff, "fused": fused, "matrices": len(shapes),
                              "ms": round(ms, 3), "matrices_per_s": round(len(shapes) / ms * 1e3, 1),
                              "tflops_algorithmic": round(alg / ms / 1e9, 1),
                              "pct_of_9pf": round(alg / ms / 1e9 / 90.0, 2),
                              "bf16_cublas_ns_loop_ms": round(bf16, 3)}), flush=True)
            del Gs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--max-size", type=int, default=16384)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--stacks", action="store_true", help="time the paper's four-block timing shapes instead")
    a = ap.parse_args()
    stream = torch.cuda.current_stream()
    if a.stacks:
        stacks(a.reps, stream)
        return
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
        if size <= 2048:
            # launch-latency-bound sizes: the same 5-iteration call replayed from a CUDA graph
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                fp4.fp4_root_ns(G, out, 5, None, ws, torch.cuda.current_stream())
            ms = _time(graph.replay, a.reps, stream)
            print(json.dumps({"case": "fp4_root_ns_graph", "size": size, "steps": 5, "ms": round(ms, 4),
                              "tflops_algorithmic": round(5 * 4.0 * size ** 3 / ms / 1e9, 1)}), flush=True)
        status = fp4.fp4_last_device_status(ws)
        assert status == 0, status
        del G, out, ws, codes, scales
        size *= 2


if __name__ == "__main__":
    main()
