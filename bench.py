#!/usr/bin/env python
"""Benchmark of the NVFP4 Root Newton-Schulz step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole hot path (clip, normalise, quantise, 5 Newton-Schulz
iterations) over the decoder-stack batch: 4 blocks x {Wq, Wk, Wv, Wo 3072x3072,
Wgate, Wup 3072x8192, Wdown 8192x3072} = 28 seeded synthetic matrices, through one
fp4_root_ns_batched call.  Prints one JSON line (rank 0).

With N > 1 (launched by torch.distributed.run) every rank runs the same batch on its own
GPU: the matrices are independent, there is no data-path collective (weak scaling).

--impl reference times the CPU oracle on the host cores on a bounded sample of the same
workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

STEPS_NS = 5
METRIC = "ns_orthogonalisations_per_s"
UNIT = "matrices/s"
FP4_NOMINAL_TFLOPS = 9000.0  # dense NVFP4, nominal
FP4_OVER_BF16 = 4.0          # nominal ratio of the dense FP4 and BF16 tensor peaks
# DRAM bytes per element of X that one G3 launch moves (dram__bytes_read + dram__bytes_write of
# k_gemm_pair<3, 0, 0, 0> from an ncu capture of one 3072 x 8192 matrix with all quantised outputs
# written: 208.6 MB for 25.2 M elements); a grouped launch is scaled by the elements it covers
G3_DRAM_BYTES_PER_ELEMENT = 208.6e6 / (3072 * 8192)
G3_KERNEL = "k_gemm_pair<3, 0, 0, 0>"   # MODE = G3, base quantiser, FP32 storage


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def batch_flops(shapes, steps=STEPS_NS):
    """(algorithmic, dense-equivalent) FLOPs of the Newton-Schulz loops of a batch."""
    alg = dense = 0.0
    for m, n in shapes:
        s, l = min(m, n), max(m, n)
        alg += steps * (3.0 * s * s * l + 1.0 * s ** 3)
        dense += steps * (4.0 * s * s * l + 2.0 * s ** 3)
    return alg, dense


def rank_seed(seed: int, rank: int) -> int:
    """Every rank draws its own batch."""
    return int(seed) + 7919 * int(rank)


def max_over_ranks(ms: float, device, world: int) -> float:
    """Step time of the job = the slowest rank's device time."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(world: int, matrices: int, steps: int, ms: float) -> float:
    """Whole-job matrices per second: every rank processed matrices * steps."""
    return world * matrices * steps / (ms / 1e3)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------
def run_reference(args):
    """The oracle as it stands, on the host cores, on a bounded sample of the batch."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2607_04422_b200 import workloads
    shapes = [(m, n) for _, m, n, _ in workloads.stack_3b_shapes(4)]
    alg_batch, _ = batch_flops(shapes)
    name, m, n, seed = workloads.stack_3b_shapes(4)[0]
    G = workloads.gradient_like(m, n, seed=seed)
    sample_steps = 1
    alg_sample, _ = batch_flops([(m, n)], steps=sample_steps)
    cores = os.cpu_count() or 1
    for _ in range(args.warmup):
        oracle.root_ns(G, steps=sample_steps)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.root_ns(G, steps=sample_steps)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    # scale the sample to the batch by its share of the algorithmic FLOPs
    batch_s = dt * alg_batch / alg_sample
    value = len(shapes) / batch_s
    sample = (f"{name} {m}x{n}, {sample_steps} of {STEPS_NS} iterations per step, scaled to the 28-matrix batch "
              f"by algorithmic FLOPs (x{alg_batch / alg_sample:.1f})")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": batch_s * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "nvfp4 operands, fp64 accumulate (CPU oracle)",
            "data": "synthetic",
            "config": {"workload": "cfg4: 3B-style decoder stack, 4 blocks x 7 projections = 28 matrices, "
                                   "5 NVFP4 Newton-Schulz iterations", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "tflops_algorithmic": alg_sample / dt / 1e12}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
def cpu_baseline_leg(mats_np, shapes):
    """Oracle on the host cores: one 3072 x 3072 matrix, all 5 iterations (about 10-30 s)."""
    import oracle
    alg_batch, _ = batch_flops(shapes)
    G = mats_np[0]
    alg_sample, _ = batch_flops([G.shape])
    t0 = time.perf_counter()
    oracle.root_ns(G, steps=STEPS_NS)
    dt = time.perf_counter() - t0
    batch_s = dt * alg_batch / alg_sample
    return {"value": len(shapes) / batch_s, "unit": UNIT, "cores": os.cpu_count() or 1, "kind": "oracle",
            "sample": f"block0.Wq {G.shape[0]}x{G.shape[1]}, 5 iterations, {dt:.1f} s; scaled to the 28-matrix "
                      f"batch by algorithmic FLOPs (x{alg_batch / alg_sample:.1f})",
            "gflops_algorithmic": alg_sample / dt / 1e9}


def small_config_rows(full_cpu: bool):
    """The single-matrix configurations measured in full on both sides: the oracle on the host cores
    (whole step, 5 iterations) and fp4_root_ns on the GPU (median of 20 calls after 5 warm-ups).  The
    256 x 512 and 2048 x 2048 cases take seconds; the 2048 x 8192 pair about a minute of host time
    and is only run with --full-cpu."""
    import torch
    import oracle
    import paper_2607_04422_b200 as fp4
    from paper_2607_04422_b200 import workloads
    cases = [("cfg1 256x512 Gaussian", workloads.config1()), ("cfg2 2048x2048 low-rank + outliers", workloads.config2())]
    if full_cpu:
        wide, tall = workloads.config3()
        cases += [("cfg3 2048x8192 row-lognormal", wide), ("cfg3 8192x2048 row-lognormal", tall)]
    rows = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, G_np in cases:
        m, n = G_np.shape
        t0 = time.perf_counter()
        want = oracle.root_ns(G_np, steps=STEPS_NS)
        cpu_s = time.perf_counter() - t0
        G = torch.from_numpy(G_np).cuda()
        out = torch.empty_like(G)
        ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(m, n, STEPS_NS), dtype=torch.uint8, device="cuda")
        times = []
        for it in range(25):
            e0.record(); fp4.fp4_root_ns(G, out, STEPS_NS, None, ws); e1.record()
            torch.cuda.synchronize()
            if it >= 5:
                times.append(e0.elapsed_time(e1))
        got = out.cpu().numpy().astype(np.float64)
        rel = float(np.linalg.norm(got - want) / np.linalg.norm(want))
        alg, _ = batch_flops([(m, n)])
        gpu_ms = float(np.median(times))
        rows.append({"workload": name, "cpu_oracle_s": cpu_s, "cpu_matrices_per_s": 1.0 / cpu_s,
                     "cpu_gflops_algorithmic": alg / cpu_s / 1e9, "gpu_ms": gpu_ms, "gpu_matrices_per_s": 1e3 / gpu_ms,
                     "gpu_tflops_algorithmic": alg / gpu_ms / 1e9, "rel_frobenius_vs_oracle": rel})
    return rows


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2607_04422_b200 as fp4
    from paper_2607_04422_b200 import workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    fp4.load_library()

    specs = workloads.stack_3b_shapes(4)
    shapes = [(m, n) for _, m, n, _ in specs]
    mats_np = [workloads.gradient_like(m, n, seed=rank_seed(seed, rank)) for _, m, n, seed in specs]
    in_bytes = sum(g.nbytes for g in mats_np)
    host_in = [torch.from_numpy(g).pin_memory() for g in mats_np]
    host_out = [torch.empty_like(h).pin_memory() for h in host_in]
    Gs = [h.cuda(non_blocking=True) for h in host_in]
    outs = [torch.empty_like(g) for g in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, STEPS_NS), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        fp4.fp4_root_ns_batched(Gs, outs, STEPS_NS, None, ws, stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    launches0 = fp4.fp4_kernel_launches()
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = fp4.fp4_kernel_launches() - launches0
    clocks = sampler.stop() if sampler else None
    status = fp4.fp4_last_device_status(ws)
    if status != 0:
        raise SystemExit(f"device status {status}: {fp4.fp4_status_string(status)}")
    # host side of one call: the call only enqueues work; timed with an empty launch queue (in the loop
    # above the host runs ahead of the GPU and mostly waits for queue space)
    host_times = []
    for _ in range(3):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        step()
        host_times.append((time.perf_counter() - t0) * 1e3)
    torch.cuda.synchronize()
    host_ms_per_call = float(np.median(host_times))
    ms = max_over_ranks(ms, torch.device("cuda"), world)
    ms_per_step = ms / args.steps
    value = aggregate_value(world, len(shapes), args.steps, ms)

    # ---- per-kernel times: one more pass with event brackets around every launch group ------
    fp4.fp4_profile_enable(True)
    prof_steps = min(args.steps, 3)
    for _ in range(prof_steps):
        step()
    torch.cuda.synchronize()
    prof = fp4.fp4_profile_collect()
    fp4.fp4_profile_enable(False)

    # ---- the same step with the paper-faithful quantiser options (random Hadamard transform of
    # every operand block and adaptive 4/6 block scaling, Section 3.4): a secondary row
    pf_params = fp4.NsParams.make(flags=fp4.FP4_FLAG_RHT | fp4.FP4_FLAG_FOUR_SIX, seed=1)
    for _ in range(2):
        fp4.fp4_root_ns_batched(Gs, outs, STEPS_NS, pf_params, ws, stream)
    torch.cuda.synchronize()
    pf_steps = min(args.steps, 5)
    e0.record(stream)
    for _ in range(pf_steps):
        fp4.fp4_root_ns_batched(Gs, outs, STEPS_NS, pf_params, ws, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    pf_ms = e0.elapsed_time(e1) / pf_steps
    if fp4.fp4_last_device_status(ws) != 0:
        raise SystemExit("device status after the paper-faithful pass")

    # ---- the same step with BF16 storage of X_k / A_k between the stages (FP4_FLAG_STORE_BF16): a secondary row
    bf_params = fp4.NsParams.make(flags=fp4.FP4_FLAG_STORE_BF16)
    ws_bf = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, STEPS_NS, fp4.FP4_FLAG_STORE_BF16),
                        dtype=torch.uint8, device="cuda")
    for _ in range(2):
        fp4.fp4_root_ns_batched(Gs, outs, STEPS_NS, bf_params, ws_bf, stream)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(pf_steps):
        fp4.fp4_root_ns_batched(Gs, outs, STEPS_NS, bf_params, ws_bf, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    bf_ms = e0.elapsed_time(e1) / pf_steps
    if fp4.fp4_last_device_status(ws_bf) != 0:
        raise SystemExit("device status after the BF16-storage pass")
    del ws_bf

    # ---- the optimiser step around it: momentum kept in the 5-bit NVFP4 state (stochastic
    # rounding), M_t = mu M_{t-1} + G_t written in FP32 together with the clip's first-pass
    # histogram, then the Root step on M_t with that histogram handed over: a secondary row
    m_codes = [torch.zeros((G.shape[0], G.shape[1] // 2), dtype=torch.uint8, device="cuda") for G in Gs]
    m_scales = [torch.zeros((G.shape[0], G.shape[1] // 16), dtype=torch.int16, device="cuda") for G in Gs]
    Ms = [torch.empty_like(G) for G in Gs]
    hists = torch.zeros((len(Gs), 8192), dtype=torch.int32, device="cuda")
    h_params = fp4.NsParams.make(top_hist=[hists[i] for i in range(len(Gs))])

    def momentum_root_step(t):
        for i, G in enumerate(Gs):
            fp4.fp4_momentum_update(G, m_codes[i], m_scales[i], Ms[i], hists[i], 0.95, 1.0, fp4.FP4_MOM_FLAG_SR,
                                    t, stream)
        fp4.fp4_root_ns_batched(Ms, outs, STEPS_NS, h_params, ws, stream)

    for t in range(2):
        momentum_root_step(t)
    torch.cuda.synchronize()
    mr_steps = min(args.steps, 5)
    e0.record(stream)
    for t in range(mr_steps):
        momentum_root_step(2 + t)
    e1.record(stream)
    torch.cuda.synchronize()
    mr_ms = e0.elapsed_time(e1) / mr_steps
    if fp4.fp4_last_device_status(ws) != 0:
        raise SystemExit("device status after the momentum + Root pass")
    # ---- and with Root's parameter update on BF16 weights: fused into the step (last product's epilogue /
    # final transpose, FP32 result not stored) against a separate update pass over the stored result
    Wts = [(torch.randn(G.shape, device="cuda") * 0.05).to(torch.bfloat16) for G in Gs]
    up_kw = dict(lr=0.02, weight_decay=0.1, update_scale=1.0)
    fused_params = fp4.NsParams.make(flags=fp4.FP4_FLAG_NO_OUT, top_hist=[hists[i] for i in range(len(Gs))],
                                     weights=Wts, **up_kw)

    def momentum_root_update_step(t, fused):
        for i, G in enumerate(Gs):
            fp4.fp4_momentum_update(G, m_codes[i], m_scales[i], Ms[i], hists[i], 0.95, 1.0, fp4.FP4_MOM_FLAG_SR,
                                    t, stream)
        if fused:
            fp4.fp4_root_ns_batched(Ms, outs, STEPS_NS, fused_params, ws, stream)
        else:
            fp4.fp4_root_ns_batched(Ms, outs, STEPS_NS, h_params, ws, stream)
            for W, o in zip(Wts, outs):      # the separate pass: W <- W * (1 - lr wd) - lr X_k in BF16
                W.mul_(1.0 - up_kw["lr"] * up_kw["weight_decay"]).add_(o, alpha=-up_kw["lr"])

    mru = {}
    for fused in (True, False):
        for t in range(2):
            momentum_root_update_step(10 + t, fused)
        torch.cuda.synchronize()
        e0.record(stream)
        for t in range(mr_steps):
            momentum_root_update_step(20 + t, fused)
        e1.record(stream)
        torch.cuda.synchronize()
        mru[fused] = e0.elapsed_time(e1) / mr_steps
    if fp4.fp4_last_device_status(ws) != 0:
        raise SystemExit("device status after the momentum + Root + update pass")
    del m_codes, m_scales, Ms, Wts

    # ---- the standalone quantiser on one 8192 x 8192 tensor (HBM-bound: 8.5625 B per element)
    qx = torch.randn((8192, 8192), device="cuda")
    qc = torch.empty((8192, 4096), dtype=torch.uint8, device="cuda")
    qs = torch.empty(fp4.fp4_scale_bytes(8192, 8192), dtype=torch.uint8, device="cuda")
    qt = torch.empty(1, device="cuda")
    q_ms = []
    for _ in range(5):
        e0.record(stream); fp4.fp4_quantize(qx, qc, qs, qt, 0, stream); e1.record(stream)
        torch.cuda.synchronize()
        q_ms.append(e0.elapsed_time(e1))
    q_gbs = 8192 * 8192 * 8.5625 / (min(q_ms[1:]) / 1e3) / 1e9
    del qx, qc, qs

    # ---- tensor-pipe ceiling of the GEMM kernel: the plain product on 8192^3 with the operands of each SM pair
    # resident in shared memory (fetched once), i.e. MMAs, commits and the FP32 epilogue only; and the same
    # product with its operand traffic
    cq = torch.empty((8192, 4096), dtype=torch.uint8, device="cuda")
    cs = torch.empty(fp4.fp4_scale_bytes(8192, 8192), dtype=torch.uint8, device="cuda")
    ct = torch.empty(1, device="cuda")
    fp4.fp4_quantize(torch.randn((8192, 8192), device="cuda"), cq, cs, ct, 0, stream)
    torch.cuda.synchronize()
    csg = float(ct.item())
    cD = torch.empty((8192, 8192), device="cuda")
    ceil = {}
    for name, fn in (("resident", fp4.fp4_gemm_nt_resident), ("streamed", fp4.fp4_gemm_nt)):
        t_ms = []
        for _ in range(6):
            e0.record(stream); fn(cq, cs, csg, cq, cs, csg, cD, None, stream); e1.record(stream)
            torch.cuda.synchronize()
            t_ms.append(e0.elapsed_time(e1))
        ceil[name] = 2.0 * 8192 ** 3 / (min(t_ms[1:]) / 1e3) / 1e12
    del cq, cs, cD

    # ---- the momentum step on one 8192 x 8192 matrix (HBM-bound: G in, M out, 5-bit state in
    # and out = 9.25 B per element), with the clip histogram and with stochastic rounding
    mg = torch.randn((8192, 8192), device="cuda")
    mm = torch.empty_like(mg)
    mc = torch.zeros((8192, 4096), dtype=torch.uint8, device="cuda")
    msc = torch.zeros((8192, 512), dtype=torch.int16, device="cuda")
    mh = torch.zeros(8192, dtype=torch.int32, device="cuda")
    mom = {}
    for name, flags in (("rtn", 0), ("sr", fp4.FP4_MOM_FLAG_SR)):
        t_ms = []
        for it in range(5):
            e0.record(stream)
            fp4.fp4_momentum_update(mg, mc, msc, mm, mh, 0.95, 1.0, flags, it, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            t_ms.append(e0.elapsed_time(e1))
        mom[name] = 8192 * 8192 * 9.25 / (min(t_ms[1:]) / 1e3) / 1e9
    del mg, mm, mc, msc

    # ---- the packed AdamW step on 2^26 BF16 parameters (both moments in NVFP4 states: 8.516 B of
    # HBM traffic per parameter), and torch's fused AdamW on FP32 tensors of the same count as context
    an = 1 << 26
    aw = (torch.randn(an, device="cuda") * 0.05).to(torch.bfloat16)
    ag = (torch.randn(an, device="cuda") * 1e-2).to(torch.bfloat16)
    amc, avc = (torch.zeros(an // 2, dtype=torch.uint8, device="cuda") for _ in range(2))
    ams, avs = (torch.zeros(an // 16, dtype=torch.int16, device="cuda") for _ in range(2))
    avm = torch.zeros(an // 256, dtype=torch.int16, device="cuda")
    adam = {}
    for name, flags in (("rtn", 0), ("sr", fp4.FP4_MOM_FLAG_SR)):
        t_ms = []
        for t in range(1, 7):
            e0.record(stream)
            fp4.fp4_adamw_update(aw, ag, amc, ams, avc, avs, avm, lr=1e-3, step=t, flags=flags, seed=t, stream=stream)
            e1.record(stream)
            torch.cuda.synchronize()
            t_ms.append(e0.elapsed_time(e1))
        adam[name] = min(t_ms[1:])
    del aw, ag, amc, avc, ams, avs, avm
    tp = torch.nn.Parameter(torch.randn(an, device="cuda") * 0.05)
    tp.grad = torch.randn(an, device="cuda") * 1e-2
    topt = torch.optim.AdamW([tp], lr=1e-3, betas=(0.9, 0.95), weight_decay=0.1, fused=True)
    t_ms = []
    for _ in range(6):
        e0.record(stream); topt.step(); e1.record(stream)
        torch.cuda.synchronize()
        t_ms.append(e0.elapsed_time(e1))
    torch_adam_ms = min(t_ms[1:])
    del tp, topt

    # ---- reference row: the same iterations in BF16 on cuBLAS (torch.matmul), dense products.
    # Context for the NVFP4 path, not part of the product.  The clip and the normalisation are
    # done once outside the timed region (torch has no fast exact quantile for 25 M elements),
    # so this row times the 15 GEMMs per matrix and their elementwise steps only.
    def bf16_prepare(G):
        X = G if G.shape[0] <= G.shape[1] else G.t()
        flat = X.abs().flatten()
        k = (990000 * flat.numel() + 999999) // 1000000
        tau = torch.kthvalue(flat, k).values
        X = X.clamp(-tau, tau)
        return (X / (X.double().norm().float() + 1e-7)).to(torch.bfloat16).contiguous()

    def bf16_ns_loop(X, abc):
        a, b, c = abc
        for _ in range(STEPS_NS):
            A = X @ X.t()
            Bm = b * A + c * (A @ A)
            X = a * X + Bm @ X
        return X

    bf16_in = [bf16_prepare(g) for g in Gs]
    bf16_abc = [fp4.fp4_root_coeffs(m, n, STEPS_NS) for m, n in shapes]
    for x, abc in list(zip(bf16_in, bf16_abc))[:3]:
        bf16_ns_loop(x, abc)
    torch.cuda.synchronize()
    e0.record(stream)
    for x, abc in zip(bf16_in, bf16_abc):
        bf16_ns_loop(x, abc)
    e1.record(stream)
    torch.cuda.synchronize()
    bf16_ms = e0.elapsed_time(e1)
    del bf16_in

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region --------
    # The batch goes through the public API one decoder block (7 matrices) at a time on three
    # streams, so that the upload of block i+1, the step on block i and the download of block
    # i-1 overlap; every byte of input and output crosses PCIe inside the timed region.
    n_blocks = 4
    per_block = len(shapes) // n_blocks
    blocks = [list(range(b * per_block, (b + 1) * per_block)) for b in range(n_blocks)]
    s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ws_blk = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes([shapes[i] for i in blocks[0]], STEPS_NS),
                         dtype=torch.uint8, device="cuda")
    ev_in = [torch.cuda.Event() for _ in blocks]
    ev_c = [torch.cuda.Event() for _ in blocks]
    ev_out = [torch.cuda.Event() for _ in blocks]
    e2e_first = [True]

    def e2e_step():
        for b, idx in enumerate(blocks):
            with torch.cuda.stream(s_in):
                if not e2e_first[0]:
                    s_in.wait_event(ev_c[b])        # the previous step has consumed these inputs
                for i in idx:
                    Gs[i].copy_(host_in[i], non_blocking=True)
                ev_in[b].record(s_in)
            with torch.cuda.stream(s_comp):
                s_comp.wait_event(ev_in[b])
                if not e2e_first[0]:
                    s_comp.wait_event(ev_out[b])    # the previous step's results have left the device
                fp4.fp4_root_ns_batched([Gs[i] for i in idx], [outs[i] for i in idx], STEPS_NS, None, ws_blk, s_comp)
                ev_c[b].record(s_comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_c[b])
                for i in idx:
                    host_out[i].copy_(outs[i], non_blocking=True)
                ev_out[b].record(s_out)
        e2e_first[0] = False

    torch.cuda.synchronize()
    e2e_step()
    barrier()
    n_e2e = max(2, min(args.steps, 5))
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(s_in)
    for _ in range(n_e2e):
        e2e_step()
    s_out.wait_stream(s_comp)
    t_end.record(s_out)
    barrier()
    e2e_ms = t_start.elapsed_time(t_end)
    assert fp4.fp4_last_device_status(ws_blk) == 0
    e2e_value = aggregate_value(world, len(shapes), n_e2e, max_over_ranks(e2e_ms, torch.device("cuda"), world))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel -----------------------------------------------------
    pk = peaks()
    alg, dense = batch_flops(shapes)
    total_prof = sum(v[0] for v in prof.values())
    shares = {k: (v[0] / total_prof if total_prof else 0.0) for k, v in prof.items()}
    dom = max(("G1", "G2", "G3"), key=lambda k: prof[k][0])
    # a launch of a stage covers a group of equal-shape matrices: compare the algorithmic
    # FLOPs of all launches of the dominant stage with the time all of them took
    flops = {"G1": 0.0, "G2": 0.0, "G3": 0.0}
    for m, n in shapes:
        s, l = min(m, n), max(m, n)
        flops["G1"] += 1.0 * s * s * l      # symmetric: half of 2 s^2 l
        flops["G2"] += 1.0 * s ** 3
        flops["G3"] += 2.0 * s * s * l
    dom_flops = flops[dom] * STEPS_NS * prof_steps      # all launches of that stage in the profiled steps
    dom_ms = prof[dom][0]
    per_launch_ms = dom_ms / max(prof[dom][1], 1)
    achieved = dom_flops / (dom_ms / 1e3) / 1e12
    fp4_peak = pk["bf16_tflops_sustained"] * FP4_OVER_BF16
    kernel_names = {"G1": "k_gemm_pair<1, 0, 0, 0>", "G2": "k_gemm_pair<2, 0, 0, 0>", "G3": G3_KERNEL}
    roofline = {"kernel": kernel_names[dom], "bound": "tensor", "achieved": achieved, "peak": fp4_peak,
                "unit": "TFLOP/s", "frac": achieved / fp4_peak,
                "traffic": (G3_DRAM_BYTES_PER_ELEMENT * sum(m * n for m, n in shapes) * STEPS_NS * prof_steps
                            / max(prof[dom][1], 1)) if dom == "G3" else None,
                "traffic_note": "DRAM bytes per launch, scaled from an ncu capture of one 3072x8192 matrix",
                "peak_source": f"{pk['source']} sustained bf16 x {FP4_OVER_BF16:.0f} (nominal FP4/BF16 ratio)",
                "avg_launch_ms": per_launch_ms, "launches_profiled": prof[dom][1],
                "flops_per_launch": dom_flops / max(prof[dom][1], 1),
                "frac_of_nominal_9pf": achieved / FP4_NOMINAL_TFLOPS,
                "mma_only_ceiling_tflops": ceil["resident"], "frac_of_mma_only_ceiling": achieved / ceil["resident"],
                "ceiling_note": "fp4_gemm_nt on 8192^3 with each SM pair's operand stages resident in shared memory "
                                "(no operand traffic): what the MMA issue, commit and FP32 epilogue of this kernel "
                                f"reach under the power cap; the same product with operand traffic: {ceil['streamed']:.0f} TFLOP/s",
                "time_share": shares}

    # the three passes of the prologue over the input (HBM-bound): bytes each moves per element of G
    n_elem = float(sum(m * n for m, n in shapes))
    pass_bytes = {"clip": 4.0, "stats": 4.0, "prep": 4.0 + 2 * 0.5625}
    prologue = {"what": "clip: histogram of the top magnitude bits + bin pick; stats: candidates of the clip bin and "
                        "sum of squares + select; prep: clamp, scale and both NVFP4 copies of X0 (no FP32 copy: "
                        "the first G3 stage reads the input itself, transposed for tall matrices)",
                "ms_per_step": sum(prof[k][0] for k in pass_bytes) / prof_steps, "passes": {}}
    for k, bpe in pass_bytes.items():
        ms_k = prof[k][0] / prof_steps
        gbs_k = n_elem * bpe / (ms_k / 1e3) / 1e9 if ms_k > 0 else 0.0
        prologue["passes"][k] = {"ms_per_step": ms_k, "bytes_per_element": bpe, "gbs": gbs_k,
                                 "frac_of_measured_hbm": gbs_k / pk["hbm_gbs"]}

    cpu = cpu_baseline_leg(mats_np, shapes)
    cpu["configs_measured_in_full"] = small_config_rows(args.full_cpu)
    step_s = ms_per_step / 1e3
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "nvfp4 operands, fp32 accumulate", "data": "synthetic",
            "config": {"workload": "cfg4: 3B-style decoder stack, 4 blocks x 7 projections = 28 matrices "
                                   "(16x 3072x3072, 8x 3072x8192, 4x 8192x3072), 5 NVFP4 Newton-Schulz iterations, "
                                   "one fp4_root_ns_batched call per step",
                       "l2": f"inputs {in_bytes / 1e9:.2f} GB per step, larger than L2; no flush needed",
                       "coefficients": "stand-in provider (the paper shows Root's values only in a figure): parity unpinned",
                       "tensor_scales": "in-loop tensor scales are predicted from running maxima (a reading of the "
                                        "paper's 'FP32 global scale'), shared by oracle and kernels",
                       "storage": "X_k and A_k kept in FP32 between the stages (headline); BF16 storage is the "
                                  "secondary row bf16_storage",
                       "parallelism": f"replicas x{world}, no collective"},
            "tflops_algorithmic": alg / step_s / 1e12, "tflops_dense_equivalent": dense / step_s / 1e12,
            "pct_of_nominal_fp4_peak": 100.0 * alg / step_s / 1e12 / FP4_NOMINAL_TFLOPS,
            "pct_of_measured_fp4_peak": 100.0 * alg / step_s / 1e12 / fp4_peak,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": in_bytes,
                    "ms_per_step": e2e_ms / n_e2e,
                    "how": "pinned host buffers; per decoder block: upload, fp4_root_ns_batched, download on three streams"},
            "quantizer": {"workload": "fp4_quantize 8192x8192 FP32", "gbs": q_gbs, "peak_gbs": pk["hbm_gbs"],
                          "frac": q_gbs / pk["hbm_gbs"], "bytes_per_element": 8.5625},
            "momentum": {"workload": "fp4_momentum_update 8192x8192 FP32 with M_t and clip histogram out",
                         "gbs": mom["rtn"], "gbs_stochastic_rounding": mom["sr"], "peak_gbs": pk["hbm_gbs"],
                         "frac": mom["rtn"] / pk["hbm_gbs"], "bytes_per_element": 9.25},
            "momentum_then_root": {"value": len(shapes) / (mr_ms / 1e3), "unit": UNIT, "ms_per_step": mr_ms,
                                   "what": "per matrix fp4_momentum_update (5-bit NVFP4 state, stochastic rounding, "
                                           "M_t and the clip histogram out), then the same batched Root step on "
                                           "M_t with the histograms handed over (the clip skips its first pass)"},
            "packed_adamw": {"workload": "fp4_adamw_update, 2^26 BF16 parameters, 42.0625 bits of state+weight+gradient "
                                         "per parameter", "us": adam["rtn"] * 1e3, "us_stochastic_rounding": adam["sr"] * 1e3,
                             "gparams_per_s": an / adam["rtn"] / 1e6, "gbs": an * 8.515625 / adam["rtn"] / 1e6,
                             "peak_gbs": pk["hbm_gbs"], "frac": an * 8.515625 / adam["rtn"] / 1e6 / pk["hbm_gbs"],
                             "bytes_per_parameter": 8.515625,
                             "torch_fused_adamw_fp32_us": torch_adam_ms * 1e3,
                             "context": "torch.optim.AdamW(fused=True) on FP32 weight, gradient and moments "
                                        "(28 B per parameter); the paper's baseline keeps BF16 weight and gradient "
                                        "with FP32 moments (22 B per parameter)"},
            "bf16_cublas_ns": {"value": len(shapes) / (bf16_ms / 1e3), "unit": UNIT, "ms_per_step": bf16_ms,
                               "tflops_dense": dense / (bf16_ms / 1e3) / 1e12,
                               "what": "the 5 Newton-Schulz iterations of the batch with torch.matmul in BF16 "
                                       "(dense, no symmetry, same coefficients); clip and normalisation outside "
                                       "the timed region; compare with our stages G1+G2+G3",
                               "our_ns_loop_ms": ms_per_step * (shares["G1"] + shares["G2"] + shares["G3"])},
            "host_ms_per_call": host_ms_per_call,
            "bf16_storage": {"value": len(shapes) / (bf_ms / 1e3), "unit": UNIT, "ms_per_step": bf_ms,
                             "what": "the same step with FP4_FLAG_STORE_BF16: X_k (k >= 1) and A_k stored in BF16 "
                                     "between the stages, operand copies and maxima still from the FP32 values"},
            "momentum_root_update": {"fused_ms_per_step": mru[True], "separate_ms_per_step": mru[False],
                                     "what": "momentum update, Root step and the BF16 parameter update of all 28 "
                                             "matrices: update fused into the step (last product's epilogue or the "
                                             "final transpose, FP32 result not stored) against the step followed "
                                             "by a separate torch pass W.mul_().add_() per matrix"},
            "rht_four_six": {"value": len(shapes) / (pf_ms / 1e3), "unit": UNIT, "ms_per_step": pf_ms,
                             "what": "the same step with FP4_FLAG_RHT | FP4_FLAG_FOUR_SIX (paper-faithful "
                                     "quantiser options); the headline value uses the base quantiser"},
            "paper_context": "paper: Root step 2.50x / 2.83x faster than optimised BF16 on one RTX 5090 (d=4096/6144)",
            "prologue": prologue,
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--full-cpu", action="store_true",
                    help="also time the oracle in full on the 2048 x 8192 pair (about a minute of host time)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
