"""fp4_quantize against the oracle: codes, scales and tensor scale bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import workloads
from paper_2607_04422_b200.binding import FP4_FLAG_FOUR_SIX, FP4_FLAG_RHT
from helpers import mismatch_report, sf_from_atoms

pytestmark = pytest.mark.gpu


def _run(x_np, flags=0):
    rows, cols = x_np.shape
    x = torch.from_numpy(x_np).cuda()
    codes = torch.empty((rows, cols // 2), dtype=torch.uint8, device="cuda")
    scales = torch.zeros(fp4.fp4_scale_bytes(rows, cols), dtype=torch.uint8, device="cuda")
    ts = torch.zeros(1, dtype=torch.float32, device="cuda")
    fp4.fp4_quantize(x, codes, scales, ts, flags=flags)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), sf_from_atoms(scales.cpu().numpy(), rows, cols // 16), float(ts.item())


def _compare(x_np):
    c, s, sg = _run(x_np)
    oc, os_, osg = oracle.quantize(x_np)
    assert np.float32(sg) == np.float32(osg)
    assert np.array_equal(s, os_), mismatch_report(s, os_)
    assert np.array_equal(c, oc), mismatch_report(c, oc)


def test_ties_saturation_and_signed_zero():
    # every E2M1 midpoint and its neighbours, E4M3 midpoints as block maxima, zeros
    f = np.float32
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], f)
    pts = np.concatenate([mids, np.nextafter(mids, f(0)), np.nextafter(mids, f(10)),
                          np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, 1e-8, 6.0], f)])
    pts = np.concatenate([pts, -pts])
    x = np.zeros((128, 128), f)
    rng = np.random.default_rng(0)
    for r in range(128):
        for b in range(8):
            blk = rng.choice(pts, 16)
            # block maximum on or next to an E4M3 rounding boundary in some rows
            top = [6.0, 6.375, 6.75, 6.0 * 1.0625, np.nextafter(f(6.375), f(7)), 5.9][(r + b) % 6]
            blk[rng.integers(16)] = top
            x[r, b * 16:(b + 1) * 16] = blk
    x[5, 16:32] = 0  # an all-zero block
    x[0, 0] = 2688.0  # tensor amax 2688 -> s_g = 1 exactly, so the ties above are hit exactly
    _compare(x * f(0.37))
    _compare(x)


@pytest.mark.parametrize("gen,shape", [
    (workloads.gaussian, (256, 512)),
    (workloads.row_lognormal, (384, 1024)),
    (workloads.lowrank_outliers, (128, 2048)),
    (workloads.gradient_like, (1024, 640)),
])
def test_workloads_bit_exact(gen, shape):
    _compare(gen(*shape, seed=3))


def test_all_zero_tensor():
    c, s, sg = _run(np.zeros((128, 128), np.float32))
    assert sg == 1.0 and not c.any() and not s.any()


def test_large_tensor_sampled_rows():
    # a tensor larger than L2; the oracle checks a sample of rows
    x = workloads.gaussian(4096, 8192, seed=5)
    c, s, sg = _run(x)
    assert np.float32(sg) == np.float32(np.abs(x).max() / np.float32(2688))
    rows = np.random.default_rng(0).choice(4096, 64, replace=False)
    oc, os_, _ = oracle.quantize(x[rows], s_g=sg)
    assert np.array_equal(c[rows], oc) and np.array_equal(s[rows], os_)


@pytest.mark.parametrize("rht,four_six", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("gen,shape", [
    (workloads.gaussian, (256, 512)),
    (workloads.row_lognormal, (384, 1024)),
    (workloads.gradient_like, (128, 4224)),     # a row is longer than one thread block covers
])
def test_paper_faithful_options_bit_exact(gen, shape, rht, four_six):
    """Random Hadamard transform and adaptive 4/6 (Section 3.4): the transform's butterfly
    order and the order of the error sums are part of the definition, so codes, block
    scales and the tensor scale agree bit for bit."""
    x = gen(*shape, seed=5)
    mask = oracle.rht_mask(17, 3) if rht else 0
    flags = (FP4_FLAG_RHT | (mask << 16) if rht else 0) | (FP4_FLAG_FOUR_SIX if four_six else 0)
    c, s, sg = _run(x, flags)
    oc, os_, osg = oracle.quantize(x, rht=rht, mask=mask, four_six=four_six)
    assert np.float32(sg) == np.float32(osg)
    assert np.array_equal(s, os_), mismatch_report(s, os_)
    assert np.array_equal(c, oc), mismatch_report(c, oc)
    if four_six:
        base = oracle.quantize(x, rht=rht, mask=mask)
        assert (s != base[1]).mean() > 0.05      # the 4-mapping is really taken


def test_paper_faithful_options_edge_blocks():
    """Blocks whose two candidate encodings tie or underflow."""
    x = np.zeros((128, 128), np.float32)
    x[0, :16] = [6, 3, 1.5, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0]        # tie: keeps the 6-mapping
    x[1, :16] = [4, 3, 2, 1, 0.5, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, -4]       # the 4-mapping is exact
    x[2, :16] = 1e-9                                                       # block scale underflows to 0
    x[3, 16:32] = np.float32(2688.0)                                       # sets the tensor scale to 1
    x[4, :16] = 5.0 / 1024                                                  # 6-scale 0, 4-scale the smallest subnormal
    c, s, sg = _run(x, FP4_FLAG_FOUR_SIX)
    oc, os_, osg = oracle.quantize(x, four_six=True)
    assert sg == osg == 1.0
    assert np.array_equal(s, os_), mismatch_report(s, os_)
    assert np.array_equal(c, oc), mismatch_report(c, oc)
    assert s[0, 0] == 0x38 and s[1, 0] == 0x38 and s[2, 0] == 0 and s[4, 0] == 1


def test_argument_errors():
    x = torch.zeros((128, 128), device="cuda")
    codes = torch.empty((128, 64), dtype=torch.uint8, device="cuda")
    scales = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    ts = torch.zeros(1, device="cuda")
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_quantize(torch.zeros((100, 128), device="cuda"), codes, scales, ts)
    assert e.value.code == 2
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_quantize(x, codes, scales, ts, flags=7)
    assert e.value.code == 1
    with pytest.raises(fp4.Fp4Error) as e:       # sign bits without the transform flag
        fp4.fp4_quantize(x, codes, scales, ts, flags=FP4_FLAG_FOUR_SIX | (0x1234 << 16))
    assert e.value.code == 1
