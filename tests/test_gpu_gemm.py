"""The tcgen05 block-scaled GEMM alone (fp4_gemm_nt) against the oracle's FP64 product."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import workloads
from helpers import sf_to_atoms

pytestmark = pytest.mark.gpu


def _dev(q):
    codes, scales, sg = q
    return (torch.from_numpy(codes).cuda(), torch.from_numpy(sf_to_atoms(scales)).cuda(), sg)


def _gemm(qa, qb):
    a, b = _dev(qa), _dev(qb)
    M, N = qa[0].shape[0], qb[0].shape[0]
    D = torch.full((M, N), float("nan"), device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    fp4.fp4_gemm_nt(a[0], a[1], a[2], b[0], b[1], b[2], D, status)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0
    return D.cpu().numpy()


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (128, 128, 512), (256, 384, 640), (640, 256, 2048),
                                   (256, 256, 256), (512, 768, 1024), (256, 512, 2048)])  # last three: CTA-pair kernel
def test_gemm_nt_matches_oracle(M, N, K):
    qa = oracle.quantize(workloads.row_lognormal(M, K, seed=1))
    qb = oracle.quantize(workloads.gaussian(N, K, seed=2))
    got = _gemm(qa, qb)
    want = oracle.gemm_nt_q(qa, qb)
    scale = np.abs(want).max()
    err = np.abs(got - want).max() / scale
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert err < 2e-6 and rel < 2e-6, (err, rel)


def test_gemm_one_hot_operands_pin_layouts():
    # A has a single non-zero block per row, B a single non-zero element per row: every
    # output is one product, so a wrong nibble order, scale position or tile mapping shows
    M = N = 256; K = 256
    a = np.zeros((M, K), np.float32); b = np.zeros((N, K), np.float32)
    rng = np.random.default_rng(0)
    for i in range(M):
        kb = i % (K // 16)
        a[i, kb * 16:(kb + 1) * 16] = rng.choice([0.5, 1, 1.5, 2, 3, 4, 6, -6, -1], 16) * 2.0 ** (i % 5)
    for j in range(N):
        b[j, (j * 7) % K] = [1.0, -2.0, 3.0, 0.5][j % 4] * 2.0 ** (j % 3)
    qa, qb = oracle.quantize(a), oracle.quantize(b)
    got = _gemm(qa, qb)
    want = oracle.gemm_nt_q(qa, qb)
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=0)
    assert np.count_nonzero(want) > 1000
