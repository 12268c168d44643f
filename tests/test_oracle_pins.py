"""Pins of the CPU oracle against things other than itself: hand-worked
fixtures, independent library codecs (ml_dtypes), closed forms, invariants,
brute force and a library SVD."""
import os

import ml_dtypes
import numpy as np
import pytest

import oracle
from paper_2607_04422_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
GRID = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], np.float64)


def _decode64(codes, scales, s_g):
    """x^ = x_E2M1 * s * s_g rebuilt from the bytes in FP64, independently of the oracle."""
    rows, cols = codes.shape[0], codes.shape[1] * 2
    nib = np.stack([codes & 0xF, codes >> 4], -1).reshape(rows, cols)
    val = np.where(nib & 8, -1.0, 1.0) * GRID[nib & 7]
    s = scales.view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    return val * np.repeat(s, 16, axis=1) * np.float64(np.float32(s_g))


def _lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [p.strip() for p in line.split("|")]


# ---- format: E2M1 and E4M3 codecs ------------------------------------------------
def test_e2m1_grid_is_the_papers():
    # Section 2: 1 sign, 2 exponent, 1 mantissa bit -> {0,.5,1,1.5,2,3,4,6}
    assert [oracle.e2m1_decode(i) for i in range(8)] == list(GRID)
    assert [oracle.e2m1_decode(8 + i) for i in range(8)] == [-v for v in GRID]


def test_e2m1_ties_and_saturation():
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for y, want in ties.items():
        assert oracle.e2m1_decode(oracle.e2m1_encode(y)) == want
        assert oracle.e2m1_decode(oracle.e2m1_encode(-y)) == -want
    for y in (6.0, 6.5, 100.0, np.inf):
        assert oracle.e2m1_encode(y) == 7 and oracle.e2m1_encode(-y) == 15
    assert oracle.e2m1_encode(-0.1) == 8  # a negative value that rounds to zero keeps its sign


def test_e2m1_encode_matches_ml_dtypes():
    rng = np.random.default_rng(0)
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], np.float32)
    pts = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(10)),
                          GRID.astype(np.float32), rng.uniform(0, 6, 4000).astype(np.float32)])
    pts = np.concatenate([pts, -pts])
    want = pts.astype(ml_dtypes.float4_e2m1fn).astype(np.float32)
    got = np.array([oracle.e2m1_decode(oracle.e2m1_encode(v)) for v in pts], np.float32)
    np.testing.assert_array_equal(got, want)


def test_ue4m3_decode_all_bytes_match_ml_dtypes():
    b = np.arange(0x7F, dtype=np.uint8)
    want = b.view(ml_dtypes.float8_e4m3fn).astype(np.float32)
    got = np.array([oracle.ue4m3_decode(int(v)) for v in b], np.float32)
    np.testing.assert_array_equal(got, want)


def test_ue4m3_encode_matches_ml_dtypes_everywhere_below_max():
    vals = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float32)
    mids = (vals[:-1].astype(np.float64) + vals[1:].astype(np.float64)) / 2  # exact in FP32
    mids = mids.astype(np.float32)
    rng = np.random.default_rng(1)
    pts = np.concatenate([vals, mids, np.nextafter(mids, np.float32(0)),
                          np.nextafter(mids, np.float32(1e9)),
                          np.exp(rng.uniform(np.log(1e-4), np.log(448), 20000)).astype(np.float32)])
    pts = pts[pts <= 448]
    want = pts.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    got = np.array([oracle.ue4m3_encode(v) for v in pts], np.uint8)
    np.testing.assert_array_equal(got, want)


def test_ue4m3_golden():
    for expr, byte, dec in _lines("ue4m3_examples.txt"):
        code = oracle.ue4m3_encode(eval(expr))
        assert code == int(byte, 16), expr
        assert oracle.ue4m3_decode(code) == eval(dec), expr


# ---- quantiser ---------------------------------------------------------------------
def test_quantiser_golden_blocks():
    for name, sg, vals, sbyte, cbytes in _lines("quantiser_examples.txt"):
        x = np.array([float(v) for v in vals.split()], np.float32).reshape(1, 16)
        codes, scales, _ = oracle.quantize(x, s_g=float(sg))
        assert scales[0, 0] == int(sbyte, 16), name
        assert [int(b) for b in codes[0]] == [int(b, 16) for b in cbytes.split()], name


def test_exact_rule_maps_tensor_amax_to_6_times_448():
    # amax 2688 -> s_g = 1, block scale 448 (0x7E), the code of 6
    name, sg, vals, sbyte, cbytes = next(l for l in _lines("quantiser_examples.txt")
                                         if l[0] == "every_tie_x448")
    x = np.array([float(v) for v in vals.split()], np.float32).reshape(1, 16)
    codes, scales, s_g = oracle.quantize(x)
    assert s_g == 1.0 and scales[0, 0] == 0x7E
    assert [int(b) for b in codes[0]] == [int(b, 16) for b in cbytes.split()]
    assert oracle.tensor_scale_exact(0.0) == 1.0


def test_fp32_operation_order_trap():
    # reciprocal-then-multiply in FP32 lands just below a tie; a division or a
    # double-precision evaluation would land on the tie and round the other way
    x = (np.arange(1, 17, dtype=np.float32) / np.float32(10)) * np.where(np.arange(16) % 2, -1, 1)
    x = x.astype(np.float32).reshape(1, 16)
    f = np.float32
    s_g = f(1.6) / f(2688)
    t = f(1.6) / (f(6) * s_g)
    assert abs(float(t) - 448) < 1e-3
    d = f(448) * s_g
    y = x[0, 1] * (f(1) / d)
    assert -0.75 < float(y) < -0.7499
    codes, scales, got_sg = oracle.quantize(x)
    assert got_sg == float(s_g) and scales[0, 0] == 0x7E
    assert (codes[0, 0] >> 4) == 9  # -0.5, not -1.0


def test_dequantisation_identity_and_error_bound():
    x = workloads.row_lognormal(64, 256, seed=3)
    codes, scales, s_g = oracle.quantize(x)
    dq = oracle.dequantize(codes, scales, s_g).astype(np.float64)
    # x^ = x_E2M1 * s * s_g, rebuilt here from the bytes
    want = _decode64(codes, scales, s_g)
    s = scales.view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    np.testing.assert_allclose(dq, want, rtol=1e-7, atol=0)
    # no block scale saturates and every block's amax stays representable
    assert scales.max() <= 0x7E
    d = np.repeat(s, 16, axis=1) * s_g
    ok = d > 0
    # error <= half the widest grid gap (1.0 -> between 4 and 6) times d, unless saturated
    err = np.abs(dq - x)[ok]
    assert np.all(err <= 1.0 * d[ok] * (1 + 1e-6) + np.abs(x)[ok] * 2.0 ** -4)


def test_quantiser_sign_symmetry_and_block_locality():
    x = workloads.gaussian(32, 128, seed=5)
    c1, s1, sg = oracle.quantize(x)
    c2, s2, _ = oracle.quantize(-x, s_g=sg)
    np.testing.assert_array_equal(s1, s2)
    np.testing.assert_array_equal(c1 ^ 0x88, c2)
    # changing one block leaves the others untouched (same global scale)
    y = x.copy(); y[3, 16:32] *= 0.5
    c3, s3, _ = oracle.quantize(y, s_g=sg)
    mask = np.ones_like(c1, bool); mask[3, 8:16] = False
    np.testing.assert_array_equal(c1[mask], c3[mask])


def test_predicted_scale_is_the_next_power_of_two():
    for bound in (2688.0, 2689.0, 1.0, 4.0, 3e-3, 1e-12, 5000.0):
        p = oracle.tensor_scale_predicted(bound)
        m, e = np.frexp(p)
        assert m == 0.5  # a power of two
        v = np.float32(bound) / np.float32(2688)
        assert p >= v and p / 2 < v
    assert oracle.tensor_scale_predicted(0.0) == 1.0


# ---- clip ----------------------------------------------------------------------------
def test_clip_threshold_worked_example():
    # |G| = {1..100}, quantile ratio 0.99 (appendix hyper-parameters) -> tau = 99
    g = np.arange(1, 101, dtype=np.float32) * np.where(np.arange(100) % 3, 1, -1)
    np.random.default_rng(0).shuffle(g)
    assert oracle.clip_threshold(g, 0.99) == 99.0
    assert oracle.quantile_rank(100, 0.99) == 99
    assert oracle.quantile_rank(4194304, 0.99) == -(-99 * 4194304 // 100)


def test_clip_threshold_brute_force():
    for seed, n in ((0, 1000), (1, 4097), (2, 16384)):
        g = np.random.default_rng(seed).standard_t(3, n).astype(np.float32)
        k = int(np.ceil(0.99 * n - 1e-9))
        want = np.sort(np.abs(g))[k - 1]
        assert oracle.clip_threshold(g, 0.99) == want
        assert np.mean(np.abs(g) > want) <= 0.01


def test_clamp_equals_input_minus_soft_threshold():
    # Section 2: soft-thresholding removes the outlier part; what is left is the clamp
    g = workloads.lowrank_outliers(128, 256, seed=2)
    out, tr = oracle.root_ns(g, steps=0, trace_iter=0)
    tau, nu = tr["tau"], tr["nu"]
    g64 = g.astype(np.float64)  # the identity is exact in FP64 (differences of FP32 numbers)
    soft = np.sign(g64) * np.maximum(np.abs(g64) - np.float64(np.float32(tau)), 0)
    clamped = (g64 - soft).astype(np.float32)
    assert np.array_equal(clamped.astype(np.float64), g64 - soft)
    assert np.abs(clamped).max() == np.float32(tau)
    nu_want = np.sqrt(np.sum(clamped.astype(np.float64) ** 2))
    assert abs(nu - nu_want) / nu_want < 1e-7
    want = clamped * (np.float32(1) / (np.float32(nu) + np.float32(1e-7)))
    np.testing.assert_array_equal(out, want)
    assert abs(np.linalg.norm(out.astype(np.float64)) - 1) < 1e-6  # Frobenius norm 1


# ---- coefficients ------------------------------------------------------------------------
def test_coefficient_identities():
    for m, n in ((512, 512), (256, 512), (2048, 8192), (8192, 2048), (3072, 8192)):
        a, b, c = oracle.root_coeffs(m, n)
        assert abs(a + b + c - 1) < 1e-6          # p(1) = 1
        assert abs(a + 3 * b + 5 * c) < 2e-6      # p'(1) = 0
        assert oracle.root_coeffs(n, m) == (a, b, c)
    a, b, c = oracle.root_coeffs(1024, 1024)
    assert (a, b, c) == (1.875, -1.25, 0.375)     # classical quintic at aspect ratio 1
    a4 = oracle.root_coeffs(2048, 8192)[0]
    a2 = oracle.root_coeffs(256, 512)[0]
    assert 1.875 < a2 < a4 < 2.1                   # wider -> steeper


# ---- Newton-Schulz ---------------------------------------------------------------------
def _poly_iter(sig, abc, k):
    a, b, c = abc
    for _ in range(k):
        sig = a * sig + b * sig ** 3 + c * sig ** 5
    return sig


@pytest.mark.parametrize("shape", [(16, 32), (48, 48), (128, 256), (96, 32)])
def test_unquantised_ns_is_the_quintic_on_singular_values(shape):
    # Section 2: X+ = aX + bX(X^T X) + cX(X^T X)^2 acts on each singular value
    g = workloads.gaussian(*shape, seed=7)
    abc = oracle.root_coeffs(*shape)
    for k in (1, 3, 5):
        out = oracle.root_ns(g, steps=k, clip_quantile=0, quantize=False)
        x0 = g.astype(np.float64) / (np.linalg.norm(g.astype(np.float64)) + 1e-7)
        U, sig, Vt = np.linalg.svd(x0, full_matrices=False)
        want = (U * _poly_iter(sig, [np.float64(np.float32(v)) for v in abc], k)) @ Vt
        err = np.linalg.norm(out - want) / np.linalg.norm(want)
        assert err < 5e-6, (k, err)


def test_tall_input_is_the_transpose_of_the_wide_one():
    g = workloads.gaussian(64, 192, seed=9)
    wide = oracle.root_ns(g, steps=3)
    tall = oracle.root_ns(np.ascontiguousarray(g.T), steps=3)
    np.testing.assert_array_equal(tall, wide.T)


def test_quantised_ns_structure():
    g = workloads.gradient_like(128, 256, seed=11)
    abc = oracle.root_coeffs(128, 256)
    out, tr = oracle.root_ns(g, steps=2, trace_iter=1)
    # A and B exactly symmetric; B = fl(fl(bA) + fl(cS)); X+ = fl(fl(aX) + P)
    np.testing.assert_array_equal(tr["A"], tr["A"].T)
    np.testing.assert_array_equal(tr["B"], tr["B"].T)
    f = np.float32
    want_B = (f(abc[1]) * tr["A"]).astype(f) + (f(abc[2]) * tr["S"]).astype(f)
    np.testing.assert_array_equal(tr["B"], want_B.astype(f))
    # each stage is the product of the decoded operands (numpy FP64 matmul as the check)
    dqX = _decode64(tr["qX_codes"], tr["qX_scales"], tr["sg_X"])
    dqXt = _decode64(tr["qXt_codes"], tr["qXt_scales"], tr["sg_X"])
    dqA = _decode64(tr["qA_codes"], tr["qA_scales"], tr["sg_A"])
    dqB = _decode64(tr["qB_codes"], tr["qB_scales"], tr["sg_B"])
    np.testing.assert_allclose(tr["A"], dqX @ dqX.T, rtol=2e-7, atol=1e-12)
    np.testing.assert_allclose(tr["S"], dqA @ dqA.T, rtol=2e-7, atol=1e-12)
    P = dqB @ dqXt.T
    want_X = (f(abc[0]) * tr["X_in"]).astype(f) + P.astype(f)
    np.testing.assert_allclose(tr["X_out"], want_X, rtol=3e-7, atol=1e-10)
    np.testing.assert_array_equal(out, tr["X_out"])
    # the two operand copies of X are quantisations of X and of its transpose
    c, s, _ = oracle.quantize(tr["X_in"], s_g=tr["sg_X"])
    np.testing.assert_array_equal(c, tr["qX_codes"]); np.testing.assert_array_equal(s, tr["qX_scales"])
    c, s, _ = oracle.quantize(np.ascontiguousarray(tr["X_in"].T), s_g=tr["sg_X"])
    np.testing.assert_array_equal(c, tr["qXt_codes"]); np.testing.assert_array_equal(s, tr["qXt_scales"])
    # predicted scales are powers of two that leave no block scale saturated
    for k in ("sg_A", "sg_B"):
        assert np.frexp(tr[k])[0] == 0.5
    for k in ("qX_scales", "qA_scales", "qB_scales"):
        assert tr[k].max() < 0x7E


def test_quantised_ns_stays_near_the_exact_iteration_and_in_the_basin():
    g = workloads.gaussian(256, 512, seed=0)
    abc = oracle.root_coeffs(256, 512)
    q = oracle.root_ns(g, steps=5, clip_quantile=0).astype(np.float64)
    e = oracle.root_ns(g, steps=5, clip_quantile=0, quantize=False).astype(np.float64)
    rel = np.linalg.norm(q - e) / np.linalg.norm(e)
    assert rel < 0.12  # NVFP4 noise floor, Section 3.4 quotes 3-10 % for such routes
    x0 = g.astype(np.float64) / np.linalg.norm(g.astype(np.float64))
    sig0 = np.linalg.svd(x0, compute_uv=False)
    lo = _poly_iter(sig0.min(), abc, 5)
    sig = np.linalg.svd(q, compute_uv=False)
    margin = 0.2636 * (1 + np.sqrt(0.5))
    assert sig.max() < 1 + margin and sig.min() > lo - margin * lo - 0.05
    # singular vectors: X close to U p^k(S) V^T of the unquantised input
    U, s0, Vt = np.linalg.svd(x0, full_matrices=False)
    want = (U * _poly_iter(s0, abc, 5)) @ Vt
    assert np.linalg.norm(q - want) / np.linalg.norm(want) < 0.12


def test_predicted_and_exact_scale_policies_have_the_same_quality():
    g = workloads.lowrank_outliers(128, 128, seed=4)
    e = oracle.root_ns(g, steps=4, quantize=False).astype(np.float64)
    p = oracle.root_ns(g, steps=4).astype(np.float64)
    x = oracle.root_ns(g, steps=4, exact_scales=True).astype(np.float64)
    ep = np.linalg.norm(p - e) / np.linalg.norm(e)
    ex = np.linalg.norm(x - e) / np.linalg.norm(e)
    assert ep < 1.5 * ex + 0.01


def test_gemm_nt_q_against_numpy():
    a = oracle.quantize(workloads.gaussian(48, 64, seed=1))
    b = oracle.quantize(workloads.gaussian(32, 64, seed=2))
    got = oracle.gemm_nt_q(a, b)
    want = _decode64(*a) @ _decode64(*b).T
    np.testing.assert_allclose(got, want, rtol=1e-7, atol=1e-7)
    sym = oracle.gemm_nt_q(a)
    np.testing.assert_array_equal(sym, sym.T)
    np.testing.assert_allclose(sym, _decode64(*a) @ _decode64(*a).T, rtol=1e-7, atol=1e-7)


# ---- paper-faithful quantiser mode: random Hadamard transform and adaptive 4/6 -----------
def _splitmix_mask(seed, idx):
    m = (1 << 64) - 1
    z = (seed + 0x9E3779B97F4A7C15 * (idx + 1)) & m
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
    z ^= z >> 31
    return z & 0xFFFF


def test_rht_mask_is_splitmix64():
    for seed, idx in ((0, 0), (1, 5), (2 ** 63 + 12345, 9), (42, 2 ** 40)):
        assert oracle.rht_mask(seed, idx) == _splitmix_mask(seed, idx)


def test_hadamard16_matches_scipy_and_is_orthonormal():
    import scipy.linalg
    H = scipy.linalg.hadamard(16).astype(np.float64) / 4.0      # natural (Sylvester) order
    eye = np.eye(16, dtype=np.float32)
    M = np.stack([oracle.hadamard16(eye[i]) for i in range(16)])  # row i = e_i H
    np.testing.assert_array_equal(M, H.astype(np.float32))
    np.testing.assert_allclose(M.astype(np.float64) @ M.astype(np.float64).T, np.eye(16), atol=1e-12)
    mask = 0b1010_0000_1111_0001
    r = np.array([-1.0 if (mask >> i) & 1 else 1.0 for i in range(16)])
    x = np.random.default_rng(0).standard_normal(16).astype(np.float32)
    np.testing.assert_allclose(oracle.hadamard16(x, mask), (x * r) @ H, rtol=1e-6, atol=1e-6)


def test_rht_cancels_in_the_product():
    # (X H)(Y H)^T = X Y^T when the same transform is applied to every 16-block along K
    rng = np.random.default_rng(1)
    X = rng.standard_normal((8, 64)).astype(np.float32)
    Y = rng.standard_normal((6, 64)).astype(np.float32)
    mask = oracle.rht_mask(7, 3)
    tx = np.stack([np.concatenate([oracle.hadamard16(row[k:k + 16], mask) for k in range(0, 64, 16)]) for row in X])
    ty = np.stack([np.concatenate([oracle.hadamard16(row[k:k + 16], mask) for k in range(0, 64, 16)]) for row in Y])
    np.testing.assert_allclose(tx.astype(np.float64) @ ty.astype(np.float64).T,
                               X.astype(np.float64) @ Y.astype(np.float64).T, rtol=0, atol=2e-5)


def test_rht_quantiser_quantises_the_transformed_blocks():
    x = workloads.gaussian(16, 128, seed=8)
    mask = oracle.rht_mask(3, 0)
    c, s, sg = oracle.quantize(x, rht=True, mask=mask)
    tx = np.stack([np.concatenate([oracle.hadamard16(row[k:k + 16], mask) for k in range(0, 128, 16)]) for row in x])
    c2, s2, _ = oracle.quantize(tx, s_g=sg)
    np.testing.assert_array_equal(c, c2)
    np.testing.assert_array_equal(s, s2)
    assert sg == oracle.tensor_scale_exact(float(np.float32(4) * np.abs(x).max()))
    assert s.max() < 0x7E


def test_four_six_golden_blocks():
    for name, vals, sbyte, cbytes in _lines("four_six_examples.txt"):
        x = np.array([float(v) for v in vals.split()], np.float32).reshape(1, 16)
        codes, scales, _ = oracle.quantize(x, s_g=1.0, four_six=True)
        assert scales[0, 0] == int(sbyte, 16), name
        assert [int(b) for b in codes[0]] == [int(b, 16) for b in cbytes.split()], name


def test_four_six_never_increases_the_block_error():
    x = workloads.row_lognormal(64, 256, seed=12)
    base = oracle.quantize(x)
    fs = oracle.quantize(x, four_six=True)
    eb = ((_decode64(*base) - x) ** 2).reshape(64, 16, 16).sum(-1)
    ef = ((_decode64(*fs) - x) ** 2).reshape(64, 16, 16).sum(-1)
    assert np.all(ef <= eb * (1 + 1e-5) + 1e-30)
    changed = fs[1] != base[1]
    assert 0.05 < changed.mean() < 0.95          # both mappings are in use
    assert ef.sum() < 0.97 * eb.sum()             # and the total error drops


@pytest.mark.parametrize("gen,shape", [(workloads.gaussian, (256, 512)), (workloads.lowrank_outliers, (256, 256))])
def test_paper_faithful_ns_is_at_least_as_close_to_exact_ns(gen, shape):
    g = gen(*shape, seed=0)
    e = oracle.root_ns(g, steps=5, quantize=False).astype(np.float64)
    base = oracle.root_ns(g, steps=5).astype(np.float64)
    pf = oracle.root_ns(g, steps=5, rht=True, four_six=True, seed=11).astype(np.float64)
    err = lambda q: np.linalg.norm(q - e) / np.linalg.norm(e)
    assert err(pf) < err(base) * 1.05
    # a different seed changes the signs, not the quality
    pf2 = oracle.root_ns(g, steps=5, rht=True, four_six=True, seed=12).astype(np.float64)
    assert not np.array_equal(pf, pf2) and abs(err(pf2) - err(pf)) < 0.03


# ---- BF16 storage of X_k and A_k between the stages ------------------------------------------
def test_bf16_round_matches_ml_dtypes():
    import ml_dtypes
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(4000).astype(np.float32) * 10.0 ** rng.integers(-20, 20, 4000),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -1e-40], np.float32)])
    # 1.00390625 = 1 + 2^-8 is a tie (rounds to even: 1.0), 1.01171875 = 1 + 3 * 2^-8 a tie that rounds up
    want = x.astype(ml_dtypes.bfloat16).astype(np.float32)
    got = oracle.bf16_round(x)
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    assert oracle.bf16_round(np.float32(1.00390625)) == 1.0 and oracle.bf16_round(np.float32(1.01171875)) == np.float32(1.015625)


def test_bf16_storage_is_a_small_perturbation_and_leaves_the_first_iteration_alone():
    g = workloads.gradient_like(256, 384, seed=2)
    base1, tr0 = oracle.root_ns(g, steps=1, trace_iter=0)
    bf1, tr1 = oracle.root_ns(g, steps=1, trace_iter=0, store_bf16=True)
    # one iteration: A is stored in BF16 (changes B), the result itself is FP32
    np.testing.assert_array_equal(tr0["A"], tr1["A"])                       # the trace holds the FP32 A
    np.testing.assert_array_equal(tr0["qA_codes"], tr1["qA_codes"])         # quantised from the FP32 values
    assert not np.array_equal(tr0["B"], tr1["B"])
    abc = oracle.root_coeffs(256, 384)
    a_st = oracle.bf16_round(tr1["A"])
    want_B = (np.float32(abc[1]) * a_st).astype(np.float32) + (np.float32(abc[2]) * tr1["S"]).astype(np.float32)
    np.testing.assert_array_equal(tr1["B"], want_B.astype(np.float32))
    e = oracle.root_ns(g, steps=5, quantize=False).astype(np.float64)
    err = lambda q: np.linalg.norm(q.astype(np.float64) - e) / np.linalg.norm(e)
    b5, f5 = oracle.root_ns(g, steps=5), oracle.root_ns(g, steps=5, store_bf16=True)
    assert abs(err(f5) - err(b5)) < 0.01 and not np.array_equal(b5, f5)
    assert f5.dtype == np.float32 and np.any(oracle.bf16_round(f5) != f5)      # the result is not rounded to BF16


@pytest.mark.parametrize("opts", [dict(), dict(rht=True, four_six=True, seed=9)])
def test_single_iteration_entry_equals_the_whole_step(opts):
    """orc_ns_iteration (one iteration from a state handed in, used to teacher-force later iterations)
    runs the same code as the loop of orc_root_ns: started from the whole step's X after iteration 0
    and the scalars the step derives there, it must return the whole step's iteration 1 bit for bit."""
    G = workloads.gradient_like(128, 384, seed=3)
    _, tr0 = oracle.root_ns(G, steps=2, trace_iter=0, **opts)
    out2, tr1 = oracle.root_ns(G, steps=2, trace_iter=1, **opts)
    X1 = tr0["X_out"]
    a = oracle.root_coeffs(128, 384)[0]
    widen = np.float32(4.0 if opts.get("rht") else 1.0)
    bound = np.float32(4.0) * np.float32(abs(a)) * np.float32(tr0["amax_in"])
    sg1 = oracle.tensor_scale_predicted(widen * bound)
    assert sg1 == tr1["sg_X"] and np.float32(np.abs(X1).max()) == np.float32(tr1["amax_in"])
    X2, amax2, sg2, tr = oracle.ns_iteration(X1, 1, tr1["amax_in"], sg1, last=True, **opts)
    assert np.array_equal(X2, out2)
    for key in ("A", "S", "B", "qA_codes", "qA_scales", "qB_codes", "qB_scales", "qX_codes", "qXt_scales"):
        assert np.array_equal(tr[key], tr1[key]), key
    assert tr["sg_A"] == tr1["sg_A"] and tr["sg_B"] == tr1["sg_B"]
    assert amax2 == np.float32(np.abs(out2).max())


# ---- Root's parameter update on BF16 weights (Section 3.4 / 3.3; the formula is a reading) -----
def _bf16(x):
    return oracle.bf16_bits(oracle.bf16_round(np.asarray(x, np.float32)))


def test_param_update_hand_worked_values():
    # w = 1, no decay, step 2^-9: 1 - 2^-9 lies halfway between the BF16 neighbours 1 - 2^-8 and 1: ties to even -> 1
    W = oracle.root_param_update(_bf16([1.0]), np.float32([1.0]), lr=2.0 ** -9, weight_decay=0.0, scale=1.0)
    assert oracle.bf16_to_f32(W)[0] == 1.0
    # a step of 3 * 2^-9 from 1: 1 - 3 * 2^-9 is halfway between 1 - 2^-7 and 1 - 2^-8: ties to even -> 1 - 2^-7
    W = oracle.root_param_update(_bf16([1.0]), np.float32([3.0]), lr=2.0 ** -9, weight_decay=0.0, scale=1.0)
    assert oracle.bf16_to_f32(W)[0] == 1.0 - 2.0 ** -7
    # decay alone: 2 * (1 - 0.5 * 0.5) = 1.5 exactly
    W = oracle.root_param_update(_bf16([2.0]), np.float32([0.0]), lr=0.5, weight_decay=0.5, scale=1.0)
    assert oracle.bf16_to_f32(W)[0] == 1.5
    # the shape factor multiplies the step: 0.25 * 4 * 0.5 = 0.5 off 3 -> 2.5
    W = oracle.root_param_update(_bf16([3.0]), np.float32([0.5]), lr=0.25, weight_decay=0.0, scale=4.0)
    assert oracle.bf16_to_f32(W)[0] == 2.5
    # sign of the step: a negative update entry raises the weight
    W = oracle.root_param_update(_bf16([0.0]), np.float32([-1.0]), lr=0.125, weight_decay=0.3, scale=1.0)
    assert oracle.bf16_to_f32(W)[0] == 0.125
    # nothing to do: lr = 0 leaves every representable weight as it is
    w0 = _bf16(np.random.default_rng(0).standard_normal(64).astype(np.float32))
    assert np.array_equal(oracle.root_param_update(w0, np.ones(64, np.float32), lr=0.0, weight_decay=0.1), w0)


def test_param_update_against_fp64():
    rng = np.random.default_rng(5)
    w = oracle.bf16_to_f32(_bf16(rng.standard_normal(4096).astype(np.float32) * 0.05))
    o = (rng.standard_normal(4096) * 0.02).astype(np.float32)
    lr, wd, sc = 0.02, 0.1, 1.6
    got = oracle.bf16_to_f32(oracle.root_param_update(_bf16(w), o, lr, wd, sc)).astype(np.float64)
    exact = w.astype(np.float64) * (1.0 - lr * wd) - lr * sc * o.astype(np.float64)
    # BF16 keeps 8 significant bits: half an ulp is at most 2^-8 of the value; the FP32 roundings add ~2^-22
    assert np.all(np.abs(got - exact) <= np.abs(exact) * (2.0 ** -8 + 2.0 ** -20) + 1e-40)
    assert np.abs(got - exact).mean() < np.abs(exact).mean() * 2.0 ** -9          # and half of that on average
    # and it is the nearest BF16 of the FP32 value the formula gives
    t = np.float32(1.0) - np.float32(lr) * np.float32(wd)
    w2 = w * t - (np.float32(lr) * np.float32(sc)) * o
    assert np.array_equal(oracle.root_param_update(_bf16(w), o, lr, wd, sc), oracle.bf16_bits(oracle.bf16_round(w2)))
