"""fp4_adamw_update against the oracle: BF16 weights and all five state arrays bit for bit, over
chained steps, with and without stochastic rounding of the first moment."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import workloads
from helpers import mismatch_report

pytestmark = pytest.mark.gpu

HP = dict(lr=2e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


def u16(t):
    return t.cpu().numpy().view(np.uint16)


class GpuAdam:
    def __init__(self, w_bits):
        n = w_bits.size
        self.W = torch.from_numpy(w_bits.view(np.int16).copy()).cuda()
        self.mc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda")
        self.ms = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
        self.vc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda")
        self.vs = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
        self.vm = torch.zeros(n // 256, dtype=torch.int16, device="cuda")

    def step(self, g_bits, t, sr=False, seed=0, **hp):
        G = torch.from_numpy(g_bits.view(np.int16).copy()).cuda()
        fp4.fp4_adamw_update(self.W, G, self.mc, self.ms, self.vc, self.vs, self.vm, step=t,
                             flags=fp4.FP4_MOM_FLAG_SR if sr else 0, seed=seed, **hp)
        torch.cuda.synchronize()

    def state(self):
        return (self.mc.cpu().numpy(), u16(self.ms), self.vc.cpu().numpy(), u16(self.vs), u16(self.vm))


def _weights(n, seed):
    return oracle.bf16_bits(workloads.gaussian(n // 256, 256, seed=seed).ravel() * np.float32(0.05))


def _grads(n, seed, scale=1e-2):
    return oracle.bf16_bits(workloads.row_lognormal(n // 256, 256, seed=seed).ravel() * np.float32(scale))


def _compare(gpu, W, st):
    assert np.array_equal(u16(gpu.W), W), mismatch_report(u16(gpu.W), W)
    names = ("m_codes", "m_scales", "v_codes", "v_scales", "v_means")
    for name, a, b in zip(names, gpu.state(), st):
        assert np.array_equal(a, b), (name, mismatch_report(a, b))


@pytest.mark.parametrize("sr", [False, True])
@pytest.mark.parametrize("n", [256, 256 * 3, 256 * 37, 256 * 1000 + 256 * 7])
def test_four_steps_bit_exact(n, sr):
    W = _weights(n, seed=n % 97)
    gpu = GpuAdam(W)
    st = None
    for t in range(1, 5):
        g = _grads(n, seed=10 * t + 1, scale=1e-2 * t)
        gpu.step(g, t, sr=sr, seed=40 + t, **HP)
        W, st, _, _ = oracle.adamw_update(W, g, st, step=t, sr=sr, seed=40 + t, **HP)
        _compare(gpu, W, st)


def test_zero_gradients_large_and_tiny_values():
    n = 256 * 8
    rng = np.random.default_rng(0)
    W = _weights(n, seed=3)
    g = np.zeros(n, np.float32)
    g[256:512] = rng.standard_normal(256) * 1e3           # large
    g[512:768] = rng.standard_normal(256) * 1e-20         # tiny: v underflows towards denormals
    g[768:1024] = 0.0                                     # a tile that never moves
    g[1024:1040] = 1.0                                    # one block of a tile
    g[1280:] = rng.standard_normal(n - 1280) * np.repeat(10.0 ** rng.integers(-6, 2, (n - 1280) // 16), 16)
    gb = oracle.bf16_bits(g)
    gpu = GpuAdam(W)
    st = None
    for t in range(1, 4):
        gpu.step(gb, t, **HP)
        W, st, _, _ = oracle.adamw_update(W, gb, st, step=t, **HP)
        _compare(gpu, W, st)
    # no weight decay, other betas
    hp = dict(lr=1e-3, beta1=0.8, beta2=0.999, eps=1e-6, weight_decay=0.0)
    gpu.step(gb, 4, sr=True, seed=5, **hp)
    W, st, _, _ = oracle.adamw_update(W, gb, st, step=4, sr=True, seed=5, **hp)
    _compare(gpu, W, st)


def test_full_size_sampled_tiles():
    # 2^26 parameters (the benchmark's size): two steps on the GPU, then tiles checked one by one
    n = 1 << 26
    gen = torch.Generator(device="cuda").manual_seed(11)
    Wt = (torch.randn(n, generator=gen, device="cuda") * 0.05).to(torch.bfloat16)
    Gs = [(torch.randn(n, generator=gen, device="cuda") * 1e-2).to(torch.bfloat16) for _ in range(2)]
    mc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda"); ms = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
    vc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda"); vs = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
    vm = torch.zeros(n // 256, dtype=torch.int16, device="cuda")
    W0 = Wt.clone()
    for t, G in enumerate(Gs, start=1):
        fp4.fp4_adamw_update(Wt, G, mc, ms, vc, vs, vm, step=t, **HP)
    torch.cuda.synchronize()
    tiles = np.sort(np.random.default_rng(1).choice(n // 256, 64, replace=False))
    idx = (torch.from_numpy(tiles).cuda()[:, None] * 256 + torch.arange(256, device="cuda")[None, :]).flatten()
    W = W0[idx].view(torch.int16).cpu().numpy().view(np.uint16)
    st = None
    for t, G in enumerate(Gs, start=1):
        W, st, _, _ = oracle.adamw_update(W, G[idx].view(torch.int16).cpu().numpy().view(np.uint16), st, step=t, **HP)
    assert np.array_equal(Wt[idx].view(torch.int16).cpu().numpy().view(np.uint16), W)
    bi = (idx.view(-1, 16)[:, 0] // 16)
    assert np.array_equal(mc.view(-1, 8)[bi].flatten().cpu().numpy(), st[0])
    assert np.array_equal(u16(ms[bi]), st[1])
    assert np.array_equal(vc.view(-1, 8)[bi].flatten().cpu().numpy(), st[2])
    assert np.array_equal(u16(vs[bi]), st[3])
    assert np.array_equal(u16(vm[torch.from_numpy(tiles).cuda()]), st[4])


def test_argument_errors():
    n = 512
    W = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    G = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    mc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda"); ms = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
    vc = torch.zeros(n // 2, dtype=torch.uint8, device="cuda"); vs = torch.zeros(n // 16, dtype=torch.int16, device="cuda")
    vm = torch.zeros(16, dtype=torch.int16, device="cuda")
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_adamw_update(W[:384], G[:384], mc, ms, vc, vs, vm, lr=1e-3)       # not a multiple of 256
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_adamw_update(W, G, mc, ms, vc, vs, vm, lr=1e-3, step=0)           # steps count from 1
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_adamw_update(W, G, mc, ms, vc, vs, vm, lr=1e-3, flags=2)          # unknown flag
    with pytest.raises(fp4.Fp4Error):
        fp4.fp4_adamw_update(W[8:264], G[:256], mc, ms, vc, vs, vm, lr=1e-3)      # W 16- but not 32-byte aligned
    fp4.fp4_adamw_update(W, G, mc, ms, vc, vs, vm, lr=1e-3)                       # and the good call works
    torch.cuda.synchronize()
