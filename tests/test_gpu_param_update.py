"""Root's parameter update fused into the step (fp4_ns_params.weights): the BF16 parameter is updated from
the orthogonalised matrix in the epilogue of the last product (CTA-pair kernel, wide or square matrix),
in the final transpose (tall matrix), or by a separate pass (single-CTA kernel shapes, no iterations,
FP4_FLAG_KEEP_OPERANDS).  All routes compute W <- BF16(fl(W*fl(1-fl(lr*wd))) - fl(fl(lr*scale)*X_k));
the oracle applies the same rule to the X_k the GPU returned, so W must agree bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import workloads
from paper_2607_04422_b200.binding import FP4_FLAG_KEEP_OPERANDS, FP4_FLAG_NO_OUT, FP4_FLAG_STORE_BF16

pytestmark = pytest.mark.gpu

LR, WD, SCALE = 0.02, 0.1, 1.4142135


def bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def make_weight(m, n, seed):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    return (torch.randn((m, n), device="cuda", generator=g) * 0.05).to(torch.bfloat16)


def run(G_np, steps, W=None, flags=0):
    m, n = G_np.shape
    G = torch.from_numpy(G_np).cuda()
    out = torch.full((m, n), float("nan"), device="cuda")
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(m, n, steps, flags), dtype=torch.uint8, device="cuda")
    p = fp4.NsParams.make(flags=flags, weights=None if W is None else [W], lr=LR, weight_decay=WD, update_scale=SCALE)
    fp4.fp4_root_ns(G, out, steps, p, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    return out


@pytest.mark.parametrize("flags", [0, FP4_FLAG_STORE_BF16, FP4_FLAG_KEEP_OPERANDS])
@pytest.mark.parametrize("shape,steps", [((512, 1024), 5), ((1024, 512), 5), ((768, 768), 3), ((384, 640), 3),
                                         ((640, 384), 2), ((512, 1024), 1), ((512, 1024), 0), ((144, 272), 3),
                                         ((400, 512), 2)])
def test_update_matches_the_oracle_rule_on_every_route(shape, steps, flags):
    m, n = shape
    G = workloads.gradient_like(m, n, seed=3)
    plain = run(G, steps, None, flags)
    W = make_weight(m, n, 1)
    w0 = bits(W).copy()
    out = run(G, steps, W, flags)
    assert torch.equal(out, plain)                              # the update does not touch the result
    want = oracle.root_param_update(w0, out.cpu().numpy(), LR, WD, SCALE)
    assert np.array_equal(bits(W), want)
    assert not np.array_equal(want, w0)
    # the update alone: same weights, the FP32 result is not stored
    W2 = make_weight(m, n, 1)
    run(G, steps, W2, flags | FP4_FLAG_NO_OUT)
    assert torch.equal(W2.view(torch.int16), W.view(torch.int16))


def test_update_in_a_batched_call_with_and_without_weights():
    specs = [(512, 1024, 1), (1024, 512, 2), (512, 1024, 3), (512, 512, 4), (384, 640, 5), (1024, 512, 6)]
    mats = [workloads.gradient_like(m, n, seed=sd) for m, n, sd in specs]
    Gs = [torch.from_numpy(g).cuda() for g in mats]
    shapes = [tuple(g.shape) for g in Gs]
    Ws = [make_weight(m, n, 10 + i) if i != 2 else None for i, (m, n, _) in enumerate(specs)]
    w0 = [None if w is None else bits(w).copy() for w in Ws]
    outs = [torch.empty_like(g) for g in Gs]
    ws = torch.empty(fp4.fp4_root_ns_batched_workspace_bytes(shapes, 4), dtype=torch.uint8, device="cuda")
    p = fp4.NsParams.make(weights=Ws, lr=LR, weight_decay=WD, update_scale=SCALE)
    fp4.fp4_root_ns_batched(Gs, outs, 4, p, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    for g, o, w, wb in zip(mats, outs, Ws, w0):
        assert torch.equal(o, run(g, 4))
        if w is not None:
            assert np.array_equal(bits(w), oracle.root_param_update(wb, o.cpu().numpy(), LR, WD, SCALE))
    # the same with the results not stored: the matrix without a weight still gets its result
    Ws2 = [make_weight(m, n, 10 + i) if i != 2 else None for i, (m, n, _) in enumerate(specs)]
    outs2 = [torch.full_like(g, float("nan")) for g in Gs]
    p2 = fp4.NsParams.make(flags=FP4_FLAG_NO_OUT, weights=Ws2, lr=LR, weight_decay=WD, update_scale=SCALE)
    fp4.fp4_root_ns_batched(Gs, outs2, 4, p2, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    assert torch.equal(outs2[2], outs[2])
    for w, w2 in zip(Ws, Ws2):
        if w is not None:
            assert torch.equal(w.view(torch.int16), w2.view(torch.int16))


@pytest.mark.parametrize("shape", [(512, 1024), (1024, 512)])
def test_two_chained_optimiser_steps_momentum_root_update(shape):
    """momentum (5-bit NVFP4 state) -> Root step on M_t -> parameter update, twice; the oracle runs the same
    chain, taking X_k from the GPU for the update (its own X_k agrees to the NS tolerance, which a BF16
    rounding may or may not hide)."""
    m, n = shape
    W = make_weight(m, n, 7)
    w_or = bits(W).copy()
    codes = torch.zeros((m, n // 2), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((m, n // 16), dtype=torch.int16, device="cuda")
    c_or = np.zeros((m, n // 2), np.uint8); s_or = np.zeros((m, n // 16), np.uint16)
    M = torch.empty((m, n), device="cuda")
    hist = torch.zeros(8192, dtype=torch.int32, device="cuda")
    out = torch.empty((m, n), device="cuda")
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(m, n, 5), dtype=torch.uint8, device="cuda")
    for t in range(2):
        G = workloads.row_lognormal(m, n, seed=40 + t)
        fp4.fp4_momentum_update(torch.from_numpy(G).cuda(), codes, scales, M, hist, 0.95, 1.0, 0, t)
        M_or, c_or, s_or, _ = oracle.momentum_update(G, c_or, s_or, 0.95, 1.0, sr=False, seed=t)
        assert np.array_equal(M.cpu().numpy(), M_or)
        p = fp4.NsParams.make(top_hist=[hist], weights=[W], lr=LR, weight_decay=WD, update_scale=SCALE)
        fp4.fp4_root_ns(M, out, 5, p, ws)
        assert fp4.fp4_last_device_status(ws) == 0
        X = out.cpu().numpy()
        ref = oracle.root_ns(M_or, steps=5).astype(np.float64)
        assert np.linalg.norm(X - ref) / np.linalg.norm(ref) <= 2e-3
        w_or = oracle.root_param_update(w_or, X, LR, WD, SCALE)
        assert np.array_equal(bits(W), w_or), t
