"""Pins of the oracle's second-moment state and packed AdamW step (Section 3.3) against things
that are not the oracle: the paper's bit count and its reconstruction claim, an exact round
trip, numpy FP64 arithmetic, the closed form of the first step and torch.optim.AdamW."""
import numpy as np
import pytest
import torch
from scipy.linalg import hadamard

import oracle

GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
H4 = hadamard(16).astype(np.float64) / 4.0


def nib_values(codes):
    c = np.asarray(codes, np.uint8)
    nib = np.empty(c.size * 2, np.uint8)
    nib[0::2] = c & 0xF
    nib[1::2] = c >> 4
    return np.where(nib & 8, -1.0, 1.0) * GRID[nib & 7]


def bf16_value(bits):
    return (np.asarray(bits, np.uint32) << 16).view(np.float32).astype(np.float64)


def numpy_v_decode(codes, scales, means):
    h = nib_values(codes).reshape(-1, 16) * bf16_value(scales)[:, None]
    r = (h @ H4).reshape(-1, 256)
    return ((r + bf16_value(means)[:, None]) ** 2).ravel()


def heavy_tailed_second_moment(n, seed):
    """EMA of squared heavy-tailed gradients with a per-group scale: non-negative, long tail."""
    rng = np.random.default_rng(seed)
    scale = np.exp(rng.standard_normal(n // 256)).repeat(256)
    v = np.zeros(n)
    for _ in range(20):
        g = rng.standard_t(4, n) * scale * 1e-3
        v = 0.95 * v + 0.05 * g * g
    return v.astype(np.float32)


def test_second_moment_is_5_0625_bits_per_element():
    # Section 3.3: 4N payload bits + N bits of per-16 BF16 scales + N/16 bits of per-256 BF16 means
    n = 256 * 12
    c, s, m = oracle.v_encode(np.ones(n, np.float32))
    assert (c.nbytes + s.nbytes + m.nbytes) * 8 == 5.0625 * n


def test_exact_round_trip():
    # sqrt-domain values mean + (grid values * 2^k) H/4 whose residuals cancel over the tile:
    # the mean is found exactly, every code is the grid value, decode returns v bit for bit
    rng = np.random.default_rng(2)
    tiles = 6
    idx = rng.integers(0, 8, (tiles, 8, 16))
    sgn = np.where(rng.integers(0, 2, (tiles, 8, 16)) == 1, -1.0, 1.0)
    idx[..., 5] = 7
    k = rng.integers(-6, -2, (tiles, 8))
    h = sgn * GRID[idx] * (2.0 ** k)[..., None]
    h = np.concatenate([h, -h], axis=1)                      # blocks 8..15 cancel blocks 0..7
    mean = (2.0 ** rng.integers(0, 3, tiles)) * 1.5          # exact in BF16, above every residual
    s = (h @ H4).reshape(tiles, 256) + mean[:, None]
    assert s.min() > 0
    v = (s * s).astype(np.float32)
    assert np.array_equal(v.astype(np.float64), s * s)       # s has few bits: the square is exact
    c, sc, m = oracle.v_encode(v.ravel())
    assert np.array_equal(bf16_value(m), mean)
    assert np.array_equal(nib_values(c).reshape(tiles, 16, 16), h / (2.0 ** np.concatenate([k, k], 1))[..., None])
    assert np.array_equal(oracle.v_decode(c, sc, m), v.ravel())


def test_mean_scales_and_decode_against_fp64():
    v = heavy_tailed_second_moment(256 * 64, seed=3)
    c, s, m = oracle.v_encode(v)
    sq = np.sqrt(v.astype(np.float64)).reshape(-1, 256)
    mean = bf16_value(m)
    # the BF16 of the FP64 mean, up to one BF16 ulp (the oracle sums in FP32)
    assert np.all(np.abs(mean - sq.mean(1)) <= sq.mean(1) * 2.0 ** -7)
    h = ((sq - mean[:, None]).reshape(-1, 16)) @ H4
    amax = np.abs(h).max(1)
    d = bf16_value(s)
    ok6 = np.abs(d - amax / 6) <= amax / 6 * 2.0 ** -7
    ok4 = np.abs(d - amax / 4) <= amax / 4 * 2.0 ** -7
    assert np.all(ok6 | ok4) and ok6.sum() > 0 and ok4.sum() > 0
    got = oracle.v_decode(c, s, m)
    want = numpy_v_decode(c, s, m)
    assert np.allclose(got, want, rtol=1e-5, atol=1e-6 * want.max())


def test_pipeline_beats_direct_nvfp4_on_a_heavy_tailed_second_moment():
    # Section 3.3, component reconstruction analysis: direct NVFP4 storage of v has about twice the
    # relative L2 error of the square root -> tile mean -> Hadamard pipeline
    v = heavy_tailed_second_moment(256 * 256, seed=4)
    c, s, m = oracle.v_encode(v)
    err_pipe = np.linalg.norm(oracle.v_decode(c, s, m) - v) / np.linalg.norm(v)
    V = v.reshape(256, 256)
    qc, qs, sg = oracle.quantize(V)
    err_direct = np.linalg.norm(oracle.dequantize(qc, qs, sg) - V) / np.linalg.norm(V)
    # in the domain the update uses (the denominator sqrt(v)), small values matter most:
    sq_pipe = np.linalg.norm(np.sqrt(oracle.v_decode(c, s, m)) - np.sqrt(v)) / np.linalg.norm(np.sqrt(v))
    sq_direct = np.linalg.norm(np.sqrt(oracle.dequantize(qc, qs, sg)).ravel() - np.sqrt(v)) / np.linalg.norm(np.sqrt(v))
    assert sq_pipe < 0.75 * sq_direct, (sq_pipe, sq_direct)
    assert err_pipe < 0.7 * err_direct, (err_pipe, err_direct)   # the paper: 0.0116 -> 0.0053 on its states


def test_first_step_closed_form():
    # zero states, t = 1: m_hat = g, v_hat = g^2, so w <- w (1 - lr wd) - lr g / (|g| + eps)
    rng = np.random.default_rng(5)
    n = 256 * 8
    w0 = oracle.bf16_to_f32(oracle.bf16_bits(rng.standard_normal(n) * 0.05))
    g = oracle.bf16_to_f32(oracle.bf16_bits(rng.standard_normal(n) * 1e-2))
    W1, st, m, v = oracle.adamw_update(oracle.bf16_bits(w0), oracle.bf16_bits(g), None, lr=2e-3, beta1=0.9,
                                       beta2=0.95, eps=1e-8, weight_decay=0.1, step=1)
    want = w0.astype(np.float64) * (1 - 2e-3 * 0.1) - 2e-3 * g / (np.abs(g) + 1e-8)
    got = oracle.bf16_to_f32(W1).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-7)     # half a BF16 ulp
    assert np.allclose(m, 0.1 * g.astype(np.float64), rtol=1e-6)
    assert np.allclose(v, 0.05 * g.astype(np.float64) ** 2, rtol=1e-6)
    # the stored states are the encodings of those moments
    mc, ms = oracle.momentum_encode(m.reshape(-1, 256))
    vc, vs, vm = oracle.v_encode(v)
    assert np.array_equal(st[0], mc.ravel()) and np.array_equal(st[1], ms.ravel())
    assert np.array_equal(st[2], vc) and np.array_equal(st[3], vs) and np.array_equal(st[4], vm)


def test_first_step_matches_torch_adamw():
    rng = np.random.default_rng(6)
    n = 256 * 4
    w0 = oracle.bf16_to_f32(oracle.bf16_bits(rng.standard_normal(n) * 0.05))
    g = oracle.bf16_to_f32(oracle.bf16_bits(rng.standard_normal(n) * 1e-2))
    p = torch.nn.Parameter(torch.from_numpy(w0.copy()))
    opt = torch.optim.AdamW([p], lr=1e-3, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.1)
    p.grad = torch.from_numpy(g.copy())
    opt.step()
    W1, _, _, _ = oracle.adamw_update(oracle.bf16_bits(w0), oracle.bf16_bits(g), None, lr=1e-3, step=1)
    got = oracle.bf16_to_f32(W1)
    want = p.detach().numpy()
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-7)


def test_several_steps_track_torch_adamw():
    # quantised states perturb the trajectory but must not bend it: after 8 steps on a fixed
    # quadratic the total displacement stays close to FP32 AdamW's
    rng = np.random.default_rng(7)
    n = 256 * 16
    target = rng.standard_normal(n).astype(np.float32) * 0.1
    w0 = oracle.bf16_to_f32(oracle.bf16_bits(rng.standard_normal(n) * 0.1))
    p = torch.nn.Parameter(torch.from_numpy(w0.copy()))
    opt = torch.optim.AdamW([p], lr=1e-2, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.0)
    W, st = oracle.bf16_bits(w0), None
    for t in range(1, 9):
        p.grad = (p.detach() - torch.from_numpy(target)).clone()
        opt.step()
        g = oracle.bf16_to_f32(W) - target
        W, st, _, _ = oracle.adamw_update(W, oracle.bf16_bits(g), st, lr=1e-2, weight_decay=0.0, step=t)
    d_ref = p.detach().numpy() - w0
    d_got = oracle.bf16_to_f32(W) - w0
    cos = float(d_ref @ d_got / (np.linalg.norm(d_ref) * np.linalg.norm(d_got)))
    assert cos > 0.95, cos      # 4-bit states: about 8 % error per stored moment
    assert abs(np.linalg.norm(d_got) / np.linalg.norm(d_ref) - 1) < 0.1


def test_update_reads_the_stored_states():
    # step 2 from stored states equals the formulas applied to the decoded states (numpy FP64)
    rng = np.random.default_rng(8)
    n = 256 * 8
    W = oracle.bf16_bits(rng.standard_normal(n) * 0.05)
    g1 = oracle.bf16_bits(rng.standard_normal(n) * 1e-2)
    g2 = oracle.bf16_bits(rng.standard_normal(n) * 1e-2)
    W1, st, _, _ = oracle.adamw_update(W, g1, None, lr=1e-3, step=1)
    W2, st2, m2, v2 = oracle.adamw_update(W1, g2, st, lr=1e-3, step=2)
    m_prev = oracle.momentum_decode(st[0].reshape(-1, 128), st[1].reshape(-1, 16)).ravel().astype(np.float64)
    v_prev = numpy_v_decode(st[2], st[3], st[4])
    g = oracle.bf16_to_f32(g2).astype(np.float64)
    m = 0.9 * m_prev + 0.1 * g
    v = 0.95 * v_prev + 0.05 * g * g
    assert np.allclose(m2, m, rtol=1e-5, atol=1e-9)
    assert np.allclose(v2, v, rtol=1e-5, atol=1e-12)
    w = oracle.bf16_to_f32(W1).astype(np.float64)
    want = w * (1 - 1e-4) - 1e-3 / (1 - 0.9 ** 2) * m / (np.sqrt(v) / np.sqrt(1 - 0.95 ** 2) + 1e-8)
    got = oracle.bf16_to_f32(W2).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-6)
