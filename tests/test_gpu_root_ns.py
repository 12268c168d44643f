"""fp4_root_ns / fp4_root_ns_batched against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import workloads
from paper_2607_04422_b200.binding import (FP4_FLAG_FOUR_SIX, FP4_FLAG_KEEP_OPERANDS, FP4_FLAG_OVERLAP_GROUPS, FP4_FLAG_RHT,
                                           FP4_FLAG_STORE_BF16,
                                           fp4_root_ns_workspace_layout)
from helpers import nibbles, sf_from_atoms

pytestmark = pytest.mark.gpu

# Tolerances.  Required of the path: relative Frobenius error of the NS output <= 2e-3 per iteration
# count, orthogonality error within 1e-2 of the oracle's.  Stage outputs that have
# bit-identical inputs on both sides differ only by FP32-vs-FP64 accumulation.
TOL_OUT = 2e-3
TOL_STAGE = 1e-5
TOL_ORTH = 1e-2


def rel(a, b):
    a = a.astype(np.float64); b = b.astype(np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def orth_err(x):
    x = x.astype(np.float64)
    if x.shape[0] > x.shape[1]:
        x = x.T
    return np.linalg.norm(x @ x.T - np.eye(x.shape[0])) / np.sqrt(x.shape[0])


def run_gpu(G_np, steps, abc=None, clip_quantile=0.99, flags=0, in_place=False, seed=0):
    m, n = G_np.shape
    G = torch.from_numpy(G_np).cuda()
    out = G if in_place else torch.full((m, n), float("nan"), device="cuda")
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(m, n, steps, flags), dtype=torch.uint8, device="cuda")
    p = fp4.NsParams.make(abc=abc, clip_quantile=clip_quantile, flags=flags, seed=seed)
    fp4.fp4_root_ns(G, out, steps, p, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    return out.cpu().numpy(), ws


def ws_view(ws, m, n, steps, flags):
    """Decodes the intermediates the last iteration left in the workspace."""
    lay = fp4_root_ns_workspace_layout(m, n, steps, flags)
    s, l = min(m, n), max(m, n)
    raw = ws.cpu().numpy()
    sc = raw[lay.scalars:lay.scalars + 4096].view(np.float32)

    def f32(off, r, c):
        return raw[off:off + r * c * 4].view(np.float32).reshape(r, c)

    def q(coff, soff, r, c):
        codes = raw[coff:coff + r * c // 2].reshape(r, c // 2)
        sf = sf_from_atoms(raw[soff:soff + r * c // 16], r, c // 16)
        return codes, sf

    return lay, sc, f32, q, s, l


QMODES = {"base": (False, False), "rht": (True, False), "four_six": (False, True), "paper": (True, True)}


def qflags(qmode):
    rht, fs = QMODES[qmode]
    return (FP4_FLAG_RHT if rht else 0) | (FP4_FLAG_FOUR_SIX if fs else 0)


@pytest.mark.parametrize("qmode", ["base", "paper", "rht", "four_six"])
@pytest.mark.parametrize("shape", [(256, 512), (384, 384), (512, 256), (128, 1152)])
def test_one_iteration_every_stage(shape, qmode):
    """Iteration 0 has bit-identical inputs on both sides: every stage is checked, in the base
    quantiser mode and with the random Hadamard transform / adaptive 4/6 of Section 3.4."""
    m, n = shape
    rht, fs = QMODES[qmode]
    seed = 99
    G = workloads.gradient_like(m, n, seed=7)
    flags = FP4_FLAG_KEEP_OPERANDS | qflags(qmode)
    got, ws = run_gpu(G, steps=1, flags=flags, seed=seed)
    want, tr = oracle.root_ns(G, steps=1, trace_iter=0, rht=rht, four_six=fs, seed=seed)
    lay, sc, f32, q, s, l = ws_view(ws, m, n, 1, flags)
    assert sc[lay.idx_nu] == np.float32(tr["nu"]), "norm differs in the last bit: pick another seed"
    assert sc[lay.idx_sg_X0] == np.float32(tr["sg_X"])
    assert sc[lay.idx_amax_X0] == np.float32(tr["amax_in"])
    # A: upper-triangle 128-tiles are stored
    A = f32(lay.A, s, s)
    mask = np.kron(np.triu(np.ones((s // 128, s // 128))), np.ones((128, 128))).astype(bool)
    assert np.abs(A[mask] - tr["A"][mask]).max() <= TOL_STAGE * np.abs(tr["A"]).max()
    assert sc[lay.idx_sg_A0] == np.float32(tr["sg_A"])
    assert abs(sc[lay.idx_amax_A0] - np.abs(tr["A"]).max()) <= 1e-6 * np.abs(tr["A"]).max()
    # qA, qB: full matrices (both triangles), a few codes may sit on rounding boundaries
    for name, co, so in (("qA", lay.qA_codes, lay.qA_scales), ("qB", lay.qB_codes, lay.qB_scales)):
        codes, sf = q(co, so, s, s)
        # blocks whose scale differs (a block amax on an E4M3 rounding boundary; with 4/6, two
        # candidate errors that nearly tie) are rare; all others agree up to codes on a boundary
        sf_diff = sf != tr[name + "_scales"]
        assert sf_diff.mean() < (6e-3 if fs else 2e-3), (name, sf_diff.mean())
        g, w = nibbles(codes), nibbles(tr[name + "_codes"])
        bad = (g != w) & ~np.repeat(sf_diff, 16, axis=1)
        assert bad.mean() < 2e-3, (name, bad.mean())
        if bad.any():
            assert np.abs((g[bad] & 7).astype(int) - (w[bad] & 7).astype(int)).max() <= 1, name
    assert sc[lay.idx_sg_B0] == np.float32(tr["sg_B"])
    # X1 and its two operand copies
    assert rel(got if m <= n else got.T, tr["X_out"]) < 2e-4
    X1 = got if m <= n else np.ascontiguousarray(got.T)
    sgX1 = sc[lay.idx_sg_X0 + 1]
    qopt = dict(rht=rht, mask=oracle.rht_mask(seed, 2) if rht else 0, four_six=fs)
    oc, os_, _ = oracle.quantize(X1, s_g=float(sgX1), **qopt)   # the GPU's own X1, quantised by the oracle
    codes, sf = q(lay.qX_codes, lay.qX_scales, s, l)
    assert np.array_equal(codes, oc) and np.array_equal(sf, os_)
    oc, os_, _ = oracle.quantize(np.ascontiguousarray(X1.T), s_g=float(sgX1), **qopt)
    codes, sf = q(lay.qXt_codes[1], lay.qXt_scales[1], l, s)
    assert np.array_equal(codes, oc) and np.array_equal(sf, os_)
    assert abs(sc[lay.idx_amax_X0 + 1] - np.abs(X1).max()) == 0


@pytest.mark.parametrize("qmode", ["base", "paper"])
@pytest.mark.parametrize("shape,gen", [((256, 512), workloads.gaussian),
                                       ((640, 384), workloads.row_lognormal),
                                       ((512, 512), workloads.lowrank_outliers)])
def test_iteration_counts_1_to_5(shape, gen, qmode):
    G = gen(*shape, seed=0)
    rht, fs = QMODES[qmode]
    for steps in (1, 2, 3, 4, 5):
        got, _ = run_gpu(G, steps=steps, flags=qflags(qmode), seed=5)
        want = oracle.root_ns(G, steps=steps, rht=rht, four_six=fs, seed=5)
        r = rel(got, want)
        assert r <= TOL_OUT, (steps, r)
        assert abs(orth_err(got) - orth_err(want)) <= TOL_ORTH


@pytest.mark.parametrize("shape", [(384, 640), (512, 1024), (1024, 512), (768, 768)])
@pytest.mark.parametrize("flags", [0, FP4_FLAG_STORE_BF16])
def test_in_place_and_determinism(shape, flags):
    """out == G, in the single-CTA kernel (384 x 640) and in the CTA-pair kernel (the others), whose
    first G3 stage reads the raw input through one tensor map while it stores X1 to the same
    addresses through another."""
    G = workloads.gradient_like(*shape, seed=5)
    a, _ = run_gpu(G, steps=3, flags=flags)
    b, _ = run_gpu(G, steps=3, flags=flags)
    c, _ = run_gpu(G.copy(), steps=3, flags=flags, in_place=True)
    assert np.array_equal(a, b) and np.array_equal(a, c)


def test_batched_in_place_pair_kernel_shapes():
    specs = [(512, 1024, 1), (1024, 512, 2), (512, 1024, 3), (512, 512, 4)]
    mats = [workloads.gradient_like(m, n, seed=sd) for m, n, sd in specs]
    Gs = [torch.from_numpy(g).cuda() for g in mats]
    shapes = [tuple(g.shape) for g in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 3), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns_batched(Gs, Gs, 3, None, ws)            # every matrix in place
    assert fp4.fp4_last_device_status(ws) == 0
    for g, o in zip(mats, Gs):
        single, _ = run_gpu(g, steps=3)
        assert np.array_equal(o.cpu().numpy(), single)


def test_tall_equals_transposed_wide():
    G = workloads.gaussian(256, 640, seed=6)
    wide, _ = run_gpu(G, steps=2)
    tall, _ = run_gpu(np.ascontiguousarray(G.T), steps=2)
    assert np.array_equal(tall, wide.T)


def test_user_coefficients():
    G = workloads.gaussian(256, 256, seed=8)
    abc = (1.6, -0.9, 0.3)
    got, _ = run_gpu(G, steps=2, abc=abc)
    want = oracle.root_ns(G, steps=2, abc=abc)
    assert rel(got, want) <= TOL_OUT


def test_batched_matches_single_calls():
    mats = workloads.stack_3b(blocks=1, scale_down=8)     # 7 matrices: 384^2, 384x1024, 1024x384
    Gs = [torch.from_numpy(g).cuda() for g in mats]
    outs = [torch.empty_like(g) for g in Gs]
    shapes = [tuple(g.shape) for g in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 5), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns_batched(Gs, outs, 5, None, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    for g, o in zip(mats, outs):
        single, _ = run_gpu(g, steps=5)
        assert np.array_equal(o.cpu().numpy(), single)
        assert rel(single, oracle.root_ns(g, steps=5)) <= TOL_OUT


def test_batched_mixed_orientations_in_one_group_paper_options():
    """Wide and tall matrices of one work shape share a lockstep group (the wide ones take
    their first FP32 tile from the raw input, the tall ones from the transposed copy); with
    the random Hadamard transform and adaptive 4/6 on, and in place for one of them."""
    specs = [(512, 256, 1), (256, 512, 2), (512, 256, 3), (256, 512, 4), (256, 256, 5)]
    mats = [workloads.gradient_like(m, n, seed=sd) for m, n, sd in specs]
    Gs = [torch.from_numpy(g).cuda() for g in mats]
    outs = [torch.empty_like(g) for g in Gs]
    outs[1] = Gs[1]                                        # in place
    shapes = [tuple(g.shape) for g in Gs]
    flags = FP4_FLAG_RHT | FP4_FLAG_FOUR_SIX
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 3, flags), dtype=torch.uint8, device="cuda")
    p = fp4.NsParams.make(flags=flags, seed=77)
    fp4.fp4_root_ns_batched(Gs, outs, 3, p, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    for g, o in zip(mats, outs):
        single, _ = run_gpu(g, steps=3, flags=flags, seed=77)
        assert np.array_equal(o.cpu().numpy(), single)
        assert rel(single, oracle.root_ns(g, steps=3, rht=True, four_six=True, seed=77)) <= TOL_OUT


@pytest.mark.parametrize("shape", [(144, 272), (272, 144), (208, 208), (16, 64), (400, 1040), (1040, 400),
                                   (496, 1008), (1008, 496)])   # the last two pad to 512 x 1024: CTA-pair kernel
def test_shapes_that_are_not_multiples_of_128(shape):
    """Dimensions that are multiples of the block length 16 are zero-padded to the tile size
    inside the library; the oracle works on the matrix as it is.  Padding must be invisible:
    the clip rank counts the caller's elements only, zero rows and columns stay zero."""
    m, n = shape
    G = workloads.gradient_like(m, n, seed=21)
    for steps in (0, 1, 3):
        got, ws = run_gpu(G, steps=steps)
        want = oracle.root_ns(G, steps=steps)
        assert got.shape == (m, n) and np.isfinite(got).all()
        assert rel(got, want) <= (1e-6 if steps == 0 else TOL_OUT), (steps, rel(got, want))
    # in place, and the two orientations agree bit for bit
    inplace, _ = run_gpu(G, steps=3, in_place=True)
    assert np.array_equal(inplace, got)
    if m != n:
        t, _ = run_gpu(np.ascontiguousarray(G.T), steps=3)
        assert np.array_equal(t.T, got)


@pytest.mark.parametrize("shape", [(128, 4096), (4096, 128), (16, 16), (16, 2048)])
def test_extreme_aspect_ratios(shape):
    m, n = shape
    G = workloads.gaussian(m, n, seed=4)
    got, _ = run_gpu(G, steps=2)
    want = oracle.root_ns(G, steps=2)
    assert rel(got, want) <= TOL_OUT, rel(got, want)


def test_largest_sweep_size_properties():
    """16384 x 16384 (the largest size of the scaling sweep, 1 GiB of FP32): no oracle run at this
    size; the result must be finite, and one iteration of the quintic must have moved the
    singular values towards 1 (the Frobenius norm of X0 is 1, so ||X1||_F > 1)."""
    size = 16384
    gen = torch.Generator(device="cuda"); gen.manual_seed(1)
    G = torch.randn((size, size), device="cuda", generator=gen)
    out = torch.empty_like(G)
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(size, size, 1), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns(G, out, 1, None, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    assert bool(torch.isfinite(out).all())
    nrm = float(out.double().norm())
    a = fp4.fp4_root_coeffs(size, size, 1)[0]
    assert 1.2 < nrm < a * 1.05, nrm          # every singular value grows by at most the slope a at zero


def test_batched_with_padded_shapes():
    specs = [(144, 272, 1), (272, 144, 2), (144, 272, 3), (256, 512, 4), (208, 208, 5)]
    mats = [workloads.gradient_like(m, n, seed=sd) for m, n, sd in specs]
    Gs = [torch.from_numpy(g).cuda() for g in mats]
    outs = [torch.full_like(g, float("nan")) for g in Gs]
    shapes = [tuple(g.shape) for g in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 4), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns_batched(Gs, outs, 4, None, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    for g, o in zip(mats, outs):
        single, _ = run_gpu(g, steps=4)
        assert np.array_equal(o.cpu().numpy(), single)
        assert rel(single, oracle.root_ns(g, steps=4)) <= TOL_OUT


def test_cuda_graph_replay_matches_direct_call():
    """The call only enqueues kernels on its stream: it can be captured in a CUDA graph
    (after one direct call has done the library's per-device set-up) and replayed."""
    G_np = workloads.config1()
    m, n = G_np.shape
    G = torch.from_numpy(G_np).cuda()
    direct = torch.empty_like(G)
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(m, n, 5), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns(G, direct, 5, None, ws)
    torch.cuda.synchronize()
    out = torch.zeros_like(G)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fp4.fp4_root_ns(G, out, 5, None, ws, torch.cuda.current_stream())
    for _ in range(2):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert fp4.fp4_last_device_status(ws) == 0
        assert torch.equal(out, direct)


def test_cuda_graph_replay_of_a_batched_call_with_several_groups():
    """With FP4_FLAG_OVERLAP_GROUPS a batched call with more than one group of shapes forks to a second
    stream and joins again: captured as a whole, the replay gives the bytes of the direct call."""
    shapes = [(256, 512), (512, 256), (512, 512), (256, 512), (768, 256), (512, 512)]
    Gs = [torch.from_numpy(workloads.gradient_like(m, n, seed=60 + i)).cuda() for i, (m, n) in enumerate(shapes)]
    direct = [torch.empty_like(x) for x in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 3), dtype=torch.uint8, device="cuda")
    p = fp4.NsParams.make(flags=FP4_FLAG_OVERLAP_GROUPS)
    fp4.fp4_root_ns_batched(Gs, direct, 3, p, ws)
    torch.cuda.synchronize()
    assert fp4.fp4_last_device_status(ws) == 0
    singles = []
    for x in Gs:
        o = torch.empty_like(x)
        w1 = torch.empty(fp4.fp4_root_ns_workspace_bytes(x.shape[0], x.shape[1], 3), dtype=torch.uint8, device="cuda")
        fp4.fp4_root_ns(x, o, 3, None, w1)
        singles.append(o)
    for a, b in zip(direct, singles):
        assert torch.equal(a, b)
    outs = [torch.zeros_like(x) for x in Gs]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fp4.fp4_root_ns_batched(Gs, outs, 3, p, ws, torch.cuda.current_stream())
    for _ in range(2):
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert fp4.fp4_last_device_status(ws) == 0
        for a, b in zip(outs, direct):
            assert torch.equal(a, b)


@pytest.mark.parametrize("shape", [(256, 512), (512, 256), (512, 512), (384, 384), (640, 384), (144, 272), (1024, 2048)])
def test_bf16_storage_of_the_high_precision_copies(shape):
    """FP4_FLAG_STORE_BF16: A_k and X_k (k >= 1) are kept in BF16 between the stages; shapes whose
    work dimensions are multiples of 256 use 2-byte tensors (CTA-pair kernel), the others FP32
    tensors with rounded values (single-CTA kernel).  Both against the oracle's emulation."""
    m, n = shape
    G = workloads.gradient_like(m, n, seed=13)
    for steps in (1, 2, 5):
        got, _ = run_gpu(G, steps=steps, flags=FP4_FLAG_STORE_BF16)
        want = oracle.root_ns(G, steps=steps, store_bf16=True)
        assert rel(got, want) <= TOL_OUT, (steps, rel(got, want))
        assert abs(orth_err(got) - orth_err(want)) <= TOL_ORTH
    plain, _ = run_gpu(G, steps=5)
    assert not np.array_equal(plain, got)                       # the option does change the numbers
    assert np.any(oracle.bf16_round(got) != got)                # the result itself is not rounded
    # iteration 0: qB is quantised from B = b bf16(A) + c S
    flags = FP4_FLAG_STORE_BF16 | FP4_FLAG_KEEP_OPERANDS
    _, ws = run_gpu(G, steps=1, flags=flags)
    _, tr = oracle.root_ns(G, steps=1, trace_iter=0, store_bf16=True)
    lay, sc, f32, q, s, l = ws_view(ws, m, n, 1, flags)
    if s % 128 == 0 and l % 128 == 0:
        codes, sf = q(lay.qB_codes, lay.qB_scales, s, s)
        sf_diff = sf != tr["qB_scales"]
        assert sf_diff.mean() < 2e-3
        g, w = nibbles(codes), nibbles(tr["qB_codes"])
        assert ((g != w) & ~np.repeat(sf_diff, 16, axis=1)).mean() < 2e-3
        raw = ws.cpu().numpy()
        if lay.Xh:   # 2-byte storage: the A region holds BF16 A (upper-triangle 128-blocks)
            A16 = raw[lay.A:lay.A + s * s * 2].view(np.uint16).reshape(s, s)
            A = (A16.astype(np.uint32) << 16).view(np.float32)
        else:
            A = f32(lay.A, s, s)
        mask = np.kron(np.triu(np.ones((s // 128, s // 128))), np.ones((128, 128))).astype(bool)
        want_A = oracle.bf16_round(tr["A"])
        # the stored A is the BF16 rounding of an FP32 value that differs from the oracle's in the last bits
        assert np.abs(A[mask] - want_A[mask]).max() <= 2.0 ** -7 * np.abs(tr["A"]).max()
        assert np.array_equal(oracle.bf16_round(A[mask]), A[mask])


def test_bf16_storage_batched_matches_single_calls():
    specs = [(256, 512, 1), (512, 256, 2), (384, 384, 3), (256, 512, 4)]
    mats = [workloads.gradient_like(m, n, seed=sd) for m, n, sd in specs]
    Gs = [torch.from_numpy(g).cuda() for g in mats]
    outs = [torch.empty_like(g) for g in Gs]
    shapes = [tuple(g.shape) for g in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 4, FP4_FLAG_STORE_BF16), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns_batched(Gs, outs, 4, fp4.NsParams.make(flags=FP4_FLAG_STORE_BF16), ws)
    assert fp4.fp4_last_device_status(ws) == 0
    for g, o in zip(mats, outs):
        single, _ = run_gpu(g, steps=4, flags=FP4_FLAG_STORE_BF16)
        assert np.array_equal(o.cpu().numpy(), single)


def test_bounded_wait_gives_up_and_reports():
    """The wait routine of the GEMM kernels, run on a barrier that nothing arrives on with a
    0.2 ms limit: it must give up, report FP4_ERR_DEVICE_TIMEOUT through the status word and
    leave the context usable (no trap, no endless spin)."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    fp4.fp4_selftest_bounded_wait(status, 200)
    torch.cuda.synchronize()
    assert int(status.item()) == 7
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_selftest_bounded_wait(status, 0)
    assert e.value.code == 1
    G = workloads.config1()
    got, _ = run_gpu(G, steps=2)                      # the context still works
    assert rel(got, oracle.root_ns(G, steps=2)) <= TOL_OUT


@pytest.mark.parametrize("shape", [(256, 512), (512, 256), (144, 272), (272, 144), (768, 1024), (400, 512)])
def test_nothing_is_written_outside_the_buffers(shape):
    """Guard regions around the workspace and the result keep their pattern (also with the
    zero padding of shapes that are not multiples of 128)."""
    m, n = shape
    G = torch.from_numpy(workloads.gradient_like(m, n, seed=9)).cuda()
    guard = 1 << 16
    need = fp4.fp4_root_ns_workspace_bytes(m, n, 3)
    big = torch.full((need + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    ws = big[guard:guard + need]
    outbig = torch.full((m * n + 2 * 4096,), 12345.0, device="cuda")
    out = outbig[4096:4096 + m * n].view(m, n)
    fp4.fp4_root_ns(G, out, 3, None, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    assert bool((big[:guard] == 0xA5).all()) and bool((big[guard + need:] == 0xA5).all())
    assert bool((outbig[:4096] == 12345.0).all()) and bool((outbig[4096 + m * n:] == 12345.0).all())
    assert rel(out.cpu().numpy(), oracle.root_ns(G.cpu().numpy(), steps=3)) <= TOL_OUT


def test_argument_errors():
    G = torch.zeros((128, 256), device="cuda")
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(128, 256, 5), dtype=torch.uint8, device="cuda")
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_root_ns(torch.zeros((100, 256), device="cuda"), G, 5, None, ws)
    assert e.value.code == 2
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_root_ns(G, G, 5, None, ws[:4096])
    assert e.value.code == 4
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_root_ns(G, G, -1, None, ws)
    assert e.value.code == 1
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_root_ns(G, G, 5, None, ws[1:])
    assert e.value.code == 3
    for bad_flags in (64, FP4_FLAG_RHT | (0x1234 << 16)):      # unknown bits, fp4_quantize's sign bits
        with pytest.raises(fp4.Fp4Error) as e:
            fp4.fp4_root_ns(G, G, 5, fp4.NsParams.make(flags=bad_flags), ws)
        assert e.value.code == 1
        with pytest.raises(fp4.Fp4Error) as e:
            fp4.fp4_root_ns_batched([G], [G], 5, fp4.NsParams.make(flags=bad_flags), ws)
        assert e.value.code == 1


# --------------------------------------------------------------------------------------
# Full-size configurations (the shapes bench.py times).  The oracle runs the whole matrix
# where that takes about a minute of host time; the iteration count is reduced for the
# largest shapes, which leaves every kernel, tile count and launch configuration unchanged.
def _full_size_case(G, steps):
    got, _ = run_gpu(G, steps=steps)
    want = oracle.root_ns(G, steps=steps)
    r = rel(got, want)
    assert r <= TOL_OUT, r
    assert abs(orth_err(got) - orth_err(want)) <= TOL_ORTH


def test_config2_square_2048_lowrank_outliers():
    _full_size_case(workloads.config2(), 5)


def test_config3_wide_and_tall_2048x8192():
    wide, tall = workloads.config3()
    _full_size_case(wide, 5)
    _full_size_case(tall, 5)


def test_config4_shapes_3072():
    specs = workloads.stack_3b_shapes(1)
    name, m, n, seed = specs[0]          # Wq 3072 x 3072
    _full_size_case(workloads.gradient_like(m, n, seed=seed), 5)
    name, m, n, seed = specs[4]          # Wgate 3072 x 8192
    _full_size_case(workloads.gradient_like(m, n, seed=seed), 3)


def test_config4_batched_full_size_properties_and_sampled_stage():
    """The 7 matrices of one decoder block at full size through fp4_root_ns_batched: the
    batched result equals the single-matrix result bit for bit, and for a wide matrix the
    first product A = qX qX^T is checked on sampled tiles that the oracle computes from its
    own clip, normalisation and quantisation of the input."""
    specs = workloads.stack_3b_shapes(1)
    mats = [workloads.gradient_like(m, n, seed=seed) for _, m, n, seed in specs]
    Gs = [torch.from_numpy(g).cuda() for g in mats]
    outs = [torch.empty_like(g) for g in Gs]
    shapes = [tuple(g.shape) for g in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 5), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns_batched(Gs, outs, 5, None, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    for idx in (0, 4, 6):                                   # 3072^2, 3072x8192, 8192x3072
        single, _ = run_gpu(mats[idx], steps=5)
        assert np.array_equal(outs[idx].cpu().numpy(), single)
        sv = np.linalg.svd(single.astype(np.float64), compute_uv=False) if idx == 0 else None
        assert np.isfinite(single).all()
        if sv is not None:
            assert sv.max() < 1.6 and sv.min() >= 0
    # sampled tiles of A (iteration 0) for the wide 3072 x 8192 matrix
    G = mats[4]
    m, n = G.shape
    flags = FP4_FLAG_KEEP_OPERANDS
    _, ws1 = run_gpu(G, steps=1, flags=flags)
    lay, sc, f32, q, s, l = ws_view(ws1, m, n, 1, flags)
    X0 = oracle.root_ns(G, steps=0)
    qx = oracle.quantize(X0)
    assert sc[lay.idx_sg_X0] == np.float32(qx[2])
    A = f32(lay.A, s, s)
    rng = np.random.default_rng(0)
    for _ in range(6):
        i = int(rng.integers(0, s // 128)); j = int(rng.integers(i, s // 128))
        rows = slice(128 * i, 128 * i + 128); cols = slice(128 * j, 128 * j + 128)
        want = oracle.gemm_nt_q((qx[0][rows], qx[1][rows], qx[2]), (qx[0][cols], qx[1][cols], qx[2]))
        assert np.abs(A[rows, cols] - want).max() <= TOL_STAGE * np.abs(want).max()


# --------------------------------------------------------------------------------------
# Degenerate inputs for the clip: so many equal magnitudes that the candidate list of the
# two-pass select overflows and the fallback passes run.
@pytest.mark.parametrize("kind", ["constant", "zero", "two_values", "ties_at_quantile"])
def test_clip_degenerate_inputs(kind):
    rng = np.random.default_rng(3)
    m, n = 256, 384
    if kind == "constant":
        G = (3.0 * rng.choice([-1.0, 1.0], (m, n))).astype(np.float32)
    elif kind == "zero":
        G = np.zeros((m, n), np.float32)
    elif kind == "two_values":
        G = rng.choice([0.5, 2.0, -2.0], (m, n)).astype(np.float32)
    else:
        G = rng.standard_normal((m, n)).astype(np.float32)
        G[np.abs(G) > 2.0] = np.float32(2.25) * np.sign(G[np.abs(G) > 2.0])   # ~4.5 % of entries tie
    got, ws = run_gpu(G, steps=0)
    want, tr = oracle.root_ns(G, steps=0, trace_iter=0)
    lay, sc, *_ = ws_view(ws, m, n, 0, 0)
    assert sc[lay.idx_tau] == np.float32(tr["tau"])
    assert abs(sc[lay.idx_nu] - tr["nu"]) <= 1.2e-7 * max(tr["nu"], 1e-30)
    assert rel(got, want) < 2e-7 or not want.any()
    if kind != "zero":
        got2, _ = run_gpu(G, steps=2)
        assert rel(got2, oracle.root_ns(G, steps=2)) <= TOL_OUT


def _first_copies_input(kind, m, n):
    rng = np.random.default_rng(1234)
    G = rng.standard_normal((m, n)).astype(np.float32)
    if kind == "dynamic_range":
        # blocks of 16 along the rows scaled by 2^-k, k up to 40: scale bytes down to the E4M3
        # subnormals and to zero, next to ordinary blocks
        k = rng.integers(0, 41, size=(m, n // 16))
        G = (G * np.repeat(np.exp2(-k), 16, axis=1)).astype(np.float32)
    elif kind == "column_dynamic_range":
        k = rng.integers(0, 41, size=(m // 16, n))
        G = (G * np.repeat(np.exp2(-k), 16, axis=0)).astype(np.float32)
    elif kind == "tiny":
        G = (G * np.float32(1e-30)).astype(np.float32)   # X0 = G / (nu + eps) stays tiny: tensor scale near 2^-90
    elif kind == "heavy_tail":
        G = (G * np.exp(2.0 * rng.standard_normal((m, n)))).astype(np.float32)
    return G


@pytest.mark.parametrize("kind", ["gaussian", "dynamic_range", "column_dynamic_range", "tiny", "heavy_tail"])
@pytest.mark.parametrize("shape", [(256, 512), (512, 256), (144, 272), (272, 144), (1024, 2048)])
def test_first_operand_copies_are_the_oracle_quantisation_of_x0(kind, shape):
    """The prologue alone (no iteration): X0 and both NVFP4 copies of it.  The copies must be, bit for bit,
    what the oracle's quantiser makes of the X0 the call returned - including blocks whose scale is an E4M3
    subnormal or zero, blocks with clipped elements, and a tensor scale far from 1."""
    m, n = shape
    G = _first_copies_input(kind, m, n)
    flags = FP4_FLAG_KEEP_OPERANDS
    got, ws = run_gpu(G, steps=0, flags=flags)
    lay, sc, f32, q, s, l = ws_view(ws, m, n, 0, flags)
    s_pad, l_pad = -(-s // 128) * 128, -(-l // 128) * 128
    X0 = np.zeros((s_pad, l_pad), dtype=np.float32)
    X0[:s, :l] = got if m <= n else got.T
    sg = float(sc[lay.idx_sg_X0])
    assert sg == np.float32(np.abs(X0).max() / np.float32(2688.0)) or np.abs(X0).max() == 0
    oc, os_, _ = oracle.quantize(X0, s_g=sg)
    codes, sf = q(lay.qX_codes, lay.qX_scales, s_pad, l_pad)
    assert np.array_equal(sf, os_), mismatch(sf, os_)
    assert np.array_equal(codes, oc), mismatch(codes, oc)
    row_scales = os_
    oc, os_, _ = oracle.quantize(np.ascontiguousarray(X0.T), s_g=sg)
    codes, sf = q(lay.qXt_codes[0], lay.qXt_scales[0], l_pad, s_pad)
    assert np.array_equal(sf, os_), mismatch(sf, os_)
    assert np.array_equal(codes, oc), mismatch(codes, oc)
    if kind in ("dynamic_range", "column_dynamic_range"):
        # the scaled blocks run along the rows of G: the copy that keeps them intact has the small scales
        along_rows = (kind == "dynamic_range") == (m <= n)
        small = row_scales if along_rows else os_
        assert ((small > 0) & (small <= 8)).any() and (small == 0).any(), "the case is meant to reach small scale bytes"


def mismatch(a, b):
    bad = np.argwhere(a != b)
    return "%d of %d differ, first at %s: %s vs %s" % (len(bad), a.size, bad[0], a[tuple(bad[0])], b[tuple(bad[0])])


@pytest.mark.parametrize("kind", ["gaussian", "heavy_tail"])
def test_first_operand_copies_two_million_blocks(kind):
    """The same on 4096 x 4096: with 2 x 10^6 blocks some scale quotients fall within two ulps of an E4M3
    rounding boundary, the case the preparation kernel hands to its exact path."""
    test_first_operand_copies_are_the_oracle_quantisation_of_x0(kind, (4096, 4096))


@pytest.mark.parametrize("qmode", ["rht", "four_six", "paper"])
@pytest.mark.parametrize("shape", [(256, 512), (512, 256), (144, 272)])
def test_first_operand_copies_with_the_paper_quantiser_options(shape, qmode):
    """The same check for the random Hadamard transform and adaptive 4/6 scaling of X0's copies (the
    transform of the first copies uses the mask of index 0; the tensor scale then covers 4 amax)."""
    m, n = shape
    rht, fs = QMODES[qmode]
    seed = 1234
    G = _first_copies_input("heavy_tail", m, n)
    flags = FP4_FLAG_KEEP_OPERANDS | qflags(qmode)
    got, ws = run_gpu(G, steps=0, flags=flags, seed=seed)
    lay, sc, f32, q, s, l = ws_view(ws, m, n, 0, flags)
    s_pad, l_pad = -(-s // 128) * 128, -(-l // 128) * 128
    X0 = np.zeros((s_pad, l_pad), dtype=np.float32)
    X0[:s, :l] = got if m <= n else got.T
    sg = float(sc[lay.idx_sg_X0])
    qopt = dict(rht=rht, mask=oracle.rht_mask(seed, 0) if rht else 0, four_six=fs)
    oc, os_, _ = oracle.quantize(X0, s_g=sg, **qopt)
    codes, sf = q(lay.qX_codes, lay.qX_scales, s_pad, l_pad)
    assert np.array_equal(sf, os_), mismatch(sf, os_)
    assert np.array_equal(codes, oc), mismatch(codes, oc)
    oc, os_, _ = oracle.quantize(np.ascontiguousarray(X0.T), s_g=sg, **qopt)
    codes, sf = q(lay.qXt_codes[0], lay.qXt_scales[0], l_pad, s_pad)
    assert np.array_equal(sf, os_), mismatch(sf, os_)
    assert np.array_equal(codes, oc), mismatch(codes, oc)


def test_two_host_threads_call_concurrently():
    """The library keeps per-thread launch state (second stream of a batched call, launch mode) and a
    locked descriptor cache: two host threads with their own streams and workspaces get the results of
    single calls."""
    import threading
    shapes = [(256, 512), (512, 256), (512, 512), (768, 256)]
    results = {}

    def worker(tid):
        torch.cuda.set_device(0)
        st = torch.cuda.Stream()
        Gs = [torch.from_numpy(workloads.gradient_like(m, n, seed=80 + 10 * tid + i)).cuda() for i, (m, n) in enumerate(shapes)]
        outs = [torch.empty_like(x) for x in Gs]
        ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 3), dtype=torch.uint8, device="cuda")
        with torch.cuda.stream(st):
            for _ in range(20):
                fp4.fp4_root_ns_batched(Gs, outs, 3, fp4.NsParams.make(flags=FP4_FLAG_OVERLAP_GROUPS), ws, st)
        st.synchronize()
        results[tid] = (Gs, outs, fp4.fp4_last_device_status(ws))

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for tid in range(2):
        Gs, outs, status = results[tid]
        assert status == 0
        for x, o in zip(Gs, outs):
            single = torch.empty_like(x)
            w1 = torch.empty(fp4.fp4_root_ns_workspace_bytes(x.shape[0], x.shape[1], 3), dtype=torch.uint8, device="cuda")
            fp4.fp4_root_ns(x, single, 3, None, w1)
            torch.cuda.synchronize()
            assert torch.equal(o, single)


@pytest.mark.parametrize("shape", [(1024, 512), (512, 1024), (1008, 496)])
def test_in_place_single_iteration(shape):
    """One iteration in place: the only G3 launch reads the caller's matrix (through a transposing box when
    it is tall) and writes the result over it."""
    m, n = shape
    G = workloads.gradient_like(m, n, seed=33)
    apart, _ = run_gpu(G, steps=1)
    inplace, _ = run_gpu(G, steps=1, in_place=True)
    assert np.array_equal(inplace, apart)
    assert rel(apart, oracle.root_ns(G, steps=1)) <= TOL_OUT
