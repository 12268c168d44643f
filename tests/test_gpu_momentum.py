"""fp4_momentum_update / fp4_momentum_decode against the oracle: M_t, codes, scales and the
histogram bit for bit, over several steps, with and without stochastic rounding."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import workloads
from helpers import mismatch_report

pytestmark = pytest.mark.gpu


class GpuState:
    def __init__(self, rows, cols):
        self.codes = torch.zeros((rows, cols // 2), dtype=torch.uint8, device="cuda")
        self.scales = torch.zeros((rows, cols // 16), dtype=torch.int16, device="cuda")

    def load(self, codes, scales):
        self.codes.copy_(torch.from_numpy(codes))
        self.scales.copy_(torch.from_numpy(scales.view(np.int16)))

    def numpy(self):
        return self.codes.cpu().numpy(), self.scales.cpu().numpy().view(np.uint16)


def _step(G_np, st, mu, g_scale=1.0, sr=False, seed=0, want_m=True, want_hist=True):
    G = torch.from_numpy(G_np).cuda()
    M = torch.empty_like(G) if want_m else None
    hist = torch.zeros(8192, dtype=torch.int32, device="cuda") if want_hist else None
    fp4.fp4_momentum_update(G, st.codes, st.scales, M, hist, mu, g_scale,
                            flags=fp4.FP4_MOM_FLAG_SR if sr else 0, seed=seed)
    torch.cuda.synchronize()
    return (M.cpu().numpy() if want_m else None,
            hist.cpu().numpy().view(np.uint32) if want_hist else None)


def _gradient(rows, cols, seed, scale=1.0):
    return (workloads.row_lognormal(rows, cols, seed=seed) * np.float32(scale)).astype(np.float32)


@pytest.mark.parametrize("sr", [False, True])
@pytest.mark.parametrize("shape", [(16, 16), (1, 4096), (48, 272), (300, 1040), (1024, 3072)])
def test_three_steps_bit_exact(shape, sr):
    rows, cols = shape
    st = GpuState(rows, cols)
    oc = np.zeros((rows, cols // 2), np.uint8)
    os_ = np.zeros((rows, cols // 16), np.uint16)
    for t in range(3):
        G = _gradient(rows, cols, seed=10 * t + rows, scale=1.0 + t)
        M, hist = _step(G, st, mu=0.95, g_scale=1.0, sr=sr, seed=77 + t)
        oM, oc, os_, oh = oracle.momentum_update(G, oc, os_, 0.95, 1.0, sr=sr, seed=77 + t)
        c, s = st.numpy()
        assert np.array_equal(M.view(np.uint32), oM.view(np.uint32)), mismatch_report(M, oM)
        assert np.array_equal(s, os_), mismatch_report(s, os_)
        assert np.array_equal(c, oc), mismatch_report(c, oc)
        assert np.array_equal(hist, oh)


def test_ema_form_and_optional_outputs():
    rows, cols = 64, 512
    G = _gradient(rows, cols, seed=3)
    st = GpuState(rows, cols)
    c0, s0 = oracle.momentum_encode(_gradient(rows, cols, seed=4))
    st.load(c0, s0)
    M, hist = _step(G, st, mu=0.9, g_scale=0.1, want_m=False, want_hist=False)
    assert M is None and hist is None
    _, oc, os_, _ = oracle.momentum_update(G, c0, s0, 0.9, 0.1)
    c, s = st.numpy()
    assert np.array_equal(c, oc) and np.array_equal(s, os_)


def test_ties_zero_blocks_and_extreme_magnitudes():
    f = np.float32
    H4 = oracle.hadamard16  # only to place chosen values in the transformed domain
    rng = np.random.default_rng(1)
    rows, cols = 32, 256
    G = np.zeros((rows, cols), f)
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 4.0, 3.0, 0.0, 0.5, 1.0, 1.5, 2.0], f)
    for r in range(rows):
        for b in range(cols // 16):
            h = rng.choice(np.concatenate([mids, -mids]), 16).astype(f)
            h[rng.integers(16)] = [6.0, 4.0, 6.0 * 1.00390625, 5.0][(r + b) % 4]
            h = h * f(2.0) ** int(rng.integers(-30, 30))
            G[r, b * 16:(b + 1) * 16] = H4(h)      # the transform is its own inverse
    G[3, 32:48] = 0
    G[4, 0:16] = f(1e-42)                          # denormals
    G[5, 16:32] = f(1e37) * np.sign(rng.standard_normal(16)).astype(f)   # sums stay finite
    G[6, 0:16] = 0
    G[6, 5] = f(-1e-30)
    for sr in (False, True):
        st = GpuState(rows, cols)
        M, hist = _step(G, st, mu=0.5, sr=sr, seed=9)
        oM, oc, os_, oh = oracle.momentum_update(G, np.zeros((rows, cols // 2), np.uint8),
                                                 np.zeros((rows, cols // 16), np.uint16), 0.5, sr=sr, seed=9)
        c, s = st.numpy()
        assert np.array_equal(M.view(np.uint32), oM.view(np.uint32))
        assert np.array_equal(s, os_), mismatch_report(s, os_)
        assert np.array_equal(c, oc), mismatch_report(c, oc)
        assert np.array_equal(hist, oh)
        # second step from that state: the decode of every such block
        G2 = np.zeros_like(G)
        M2, _ = _step(G2, st, mu=1.0, sr=sr, seed=10)
        oM2, _, _, _ = oracle.momentum_update(G2, oc, os_, 1.0, sr=sr, seed=10)
        assert np.array_equal(M2.view(np.uint32), oM2.view(np.uint32))


def test_decode_entry_point():
    rows, cols = 96, 784
    c0, s0 = oracle.momentum_encode(_gradient(rows, cols, seed=12))
    st = GpuState(rows, cols)
    st.load(c0, s0)
    M = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
    fp4.fp4_momentum_decode(st.codes, st.scales, M)
    torch.cuda.synchronize()
    assert np.array_equal(M.cpu().numpy().view(np.uint32), oracle.momentum_decode(c0, s0).view(np.uint32))
    c, s = st.numpy()
    assert np.array_equal(c, c0) and np.array_equal(s, s0)


def test_full_size_sampled_rows_and_histogram():
    # the benchmark's size: rows checked one by one against the oracle, the histogram against the
    # kernel's own M_t
    rows, cols = 8192, 8192
    gen = torch.Generator(device="cuda").manual_seed(5)
    G = torch.randn((rows, cols), generator=gen, device="cuda", dtype=torch.float32)
    G *= torch.exp(0.5 * torch.randn((rows, 1), generator=gen, device="cuda"))
    st = GpuState(rows, cols)
    M = torch.empty_like(G)
    hist = torch.zeros(8192, dtype=torch.int32, device="cuda")
    for t in range(2):
        prev_c, prev_s = st.codes.clone(), st.scales.clone()
        hist.zero_()
        fp4.fp4_momentum_update(G, st.codes, st.scales, M, hist, 0.95, 1.0, flags=fp4.FP4_MOM_FLAG_SR, seed=t)
    torch.cuda.synchronize()
    assert int(hist.sum().item()) == rows * cols
    bins = (M.view(torch.int32) & 0x7FFFFFFF) >> 18
    want = torch.bincount(bins.flatten().long(), minlength=8192)
    assert torch.equal(want.to(torch.int32), hist)
    # without stochastic rounding any row can be checked alone; with it the random stream is
    # numbered by matrix position, so the leading rows are
    head = 8
    oM, oc, os_, _ = oracle.momentum_update(G[:head].cpu().numpy(), prev_c[:head].cpu().numpy(),
                                            prev_s[:head].cpu().numpy().view(np.uint16), 0.95, 1.0, sr=True, seed=1)
    assert np.array_equal(M[:head].cpu().numpy().view(np.uint32), oM.view(np.uint32))
    assert np.array_equal(st.codes[:head].cpu().numpy(), oc)
    assert np.array_equal(st.scales[:head].cpu().numpy().view(np.uint16), os_)
    idx = torch.tensor(np.random.default_rng(0).choice(rows, 24, replace=False), device="cuda")
    Gs = G[idx].cpu().numpy()
    pc, ps = prev_c[idx].cpu().numpy(), prev_s[idx].cpu().numpy().view(np.uint16)
    st2_c, st2_s = prev_c.clone(), prev_s.clone()
    fp4.fp4_momentum_update(G, st2_c, st2_s, M, None, 0.95, 1.0)
    torch.cuda.synchronize()
    oM, oc, os_, _ = oracle.momentum_update(Gs, pc, ps, 0.95, 1.0)
    assert np.array_equal(M[idx].cpu().numpy().view(np.uint32), oM.view(np.uint32))
    assert np.array_equal(st2_c[idx].cpu().numpy(), oc)
    assert np.array_equal(st2_s[idx].cpu().numpy().view(np.uint16), os_)


def test_argument_errors():
    G = torch.zeros((16, 24), dtype=torch.float32, device="cuda")
    c = torch.zeros((16, 12), dtype=torch.uint8, device="cuda")
    s = torch.zeros((16, 2), dtype=torch.int16, device="cuda")
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_momentum_update(G, c, s, None, None, 0.9)            # cols not a multiple of 16
    G = torch.zeros((16, 32), dtype=torch.float32, device="cuda")
    c = torch.zeros((16, 16), dtype=torch.uint8, device="cuda")
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_momentum_update(G, c, s, None, None, 0.9, flags=4)   # unknown flag
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_momentum_update(G.flatten()[1:].reshape(1, -1)[:, :16], c, s, None, None, 0.9)  # misaligned
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_momentum_update(G.flatten()[4:].reshape(1, -1)[:, :16], c, s, None, None, 0.9)  # 16 but not 32 bytes


def _ns(G, steps=2, top_hist=None):
    m, n = G.shape
    out = torch.full((m, n), float("nan"), device="cuda")
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(m, n, steps, 0), dtype=torch.uint8, device="cuda")
    p = fp4.NsParams.make(top_hist=top_hist)
    fp4.fp4_root_ns(G, out, steps, p, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    return out


@pytest.mark.parametrize("shape", [(256, 512), (1024, 384), (400, 1136)])
def test_momentum_histogram_feeds_the_clip(shape):
    # M_t and its histogram from the momentum step; the Newton-Schulz step that takes the
    # histogram must give exactly what it gives when it counts M_t itself, and the oracle chain
    # (momentum step, then Root step) must agree with the GPU chain
    rows, cols = shape
    G = _gradient(rows, cols, seed=21)
    st = GpuState(rows, cols)
    c0, s0 = oracle.momentum_encode(_gradient(rows, cols, seed=22))
    st.load(c0, s0)
    Gd = torch.from_numpy(G).cuda()
    M = torch.empty_like(Gd)
    hist = torch.zeros(8192, dtype=torch.int32, device="cuda")
    fp4.fp4_momentum_update(Gd, st.codes, st.scales, M, hist, 0.95, 1.0)
    ref = _ns(M)
    got = _ns(M, top_hist=[hist])
    torch.cuda.synchronize()
    assert torch.equal(ref, got)
    assert int(hist.abs().sum().item()) == 0          # consumed
    oM, _, _, _ = oracle.momentum_update(G, c0, s0, 0.95, 1.0)
    assert np.array_equal(M.cpu().numpy().view(np.uint32), oM.view(np.uint32))
    want = oracle.root_ns(oM, 2)
    err = np.linalg.norm(got.cpu().numpy() - want) / np.linalg.norm(want)
    assert err < 2e-3, err


def test_momentum_histograms_in_a_batched_call():
    shapes = [(256, 512), (256, 512), (512, 256), (384, 384), (256, 512)]
    Ms, hists, outs_ref = [], [], []
    for i, (r, c) in enumerate(shapes):
        Gd = torch.from_numpy(_gradient(r, c, seed=30 + i)).cuda()
        st = GpuState(r, c)
        M = torch.empty_like(Gd)
        h = torch.zeros(8192, dtype=torch.int32, device="cuda")
        fp4.fp4_momentum_update(Gd, st.codes, st.scales, M, h, 0.9, 1.0)
        Ms.append(M)
        hists.append(h if i != 1 else None)           # one matrix of a group counts for itself
        outs_ref.append(_ns(M, steps=3))
    outs = [torch.empty_like(M) for M in Ms]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 3, 0), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns_batched(Ms, outs, 3, fp4.NsParams.make(top_hist=hists), ws)
    assert fp4.fp4_last_device_status(ws) == 0
    for a, b in zip(outs, outs_ref):
        assert torch.equal(a, b)
    for h in hists:
        if h is not None:
            assert int(h.abs().sum().item()) == 0


def test_optimizer_chain_in_a_cuda_graph():
    """Momentum step, Root step with the histogram handed over and a packed AdamW step only
    enqueue kernels on their stream: the chain is captured once and replayed on new gradients."""
    rows, cols = 256, 512
    n = rows * cols
    G = torch.empty((rows, cols), device="cuda")
    Gb = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    st = GpuState(rows, cols)
    M = torch.empty_like(G)
    hist = torch.zeros(8192, dtype=torch.int32, device="cuda")
    out = torch.empty_like(G)
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(rows, cols, 3), dtype=torch.uint8, device="cuda")
    W = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    mc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda"); ms = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
    vc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda"); vs = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
    vm = torch.zeros(n // 256, dtype=torch.int16, device="cuda")
    prm = fp4.NsParams.make(top_hist=[hist])

    def chain(stream=None):
        fp4.fp4_momentum_update(G, st.codes, st.scales, M, hist, 0.95, 1.0, stream=stream)
        fp4.fp4_root_ns(M, out, 3, prm, ws, stream)
        fp4.fp4_adamw_update(W, Gb, mc, ms, vc, vs, vm, lr=1e-3, step=1, stream=stream)

    G.copy_(torch.from_numpy(_gradient(rows, cols, seed=50)))
    Gb.copy_(G.flatten().to(torch.bfloat16))
    chain()                                   # per-device set-up happens outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        chain(torch.cuda.current_stream())
    # oracle mirror of the replays, starting from the states the direct call and the capture left
    # (a capture does not execute anything)
    oc, os_ = st.numpy()
    oW = W.view(torch.int16).cpu().numpy().view(np.uint16)
    ost = (mc.cpu().numpy(), ms.cpu().numpy().view(np.uint16), vc.cpu().numpy(), vs.cpu().numpy().view(np.uint16),
           vm.cpu().numpy().view(np.uint16))
    for rep in range(2):
        g_np = _gradient(rows, cols, seed=60 + rep)
        G.copy_(torch.from_numpy(g_np))
        Gb.copy_(G.flatten().to(torch.bfloat16))
        graph.replay()
        torch.cuda.synchronize()
        assert fp4.fp4_last_device_status(ws) == 0
        oM, oc, os_, _ = oracle.momentum_update(g_np, oc, os_, 0.95, 1.0)
        assert np.array_equal(M.cpu().numpy().view(np.uint32), oM.view(np.uint32))
        c, s = st.numpy()
        assert np.array_equal(c, oc) and np.array_equal(s, os_)
        want = oracle.root_ns(oM, 3)
        err = np.linalg.norm(out.cpu().numpy() - want) / np.linalg.norm(want)
        assert err < 2e-3, err
        assert int(hist.abs().sum().item()) == 0
        gb = Gb.view(torch.int16).cpu().numpy().view(np.uint16)
        oW, ost, _, _ = oracle.adamw_update(oW, gb, ost, lr=1e-3, step=1)
        assert np.array_equal(W.view(torch.int16).cpu().numpy().view(np.uint16), oW)
