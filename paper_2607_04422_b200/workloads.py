"""Seeded synthetic inputs shaped like the update matrices the Root step sees.

This module holds no arithmetic of the method (no quantisation, clipping,
normalisation or Newton-Schulz): it only draws random matrices.  It serves the
CUDA library's tests and benchmark and the CPU oracle's tests alike, so that
"the same seeded inputs" is literal.  Everything is generated on the host with
numpy's counter-based Philox generator and returned as C-contiguous FP32.

The paper's own inputs are gradient/momentum matrices of a decoder being
trained (Section 4.1); those are not available, so each workload below keeps the
properties that matter to the step: the projection shapes of a decoder block,
a low-rank component, and a sparse set of heavy-tailed outliers that the p99
clip is there to remove (Section 3.4).
"""
from __future__ import annotations

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(int(seed)))


def gaussian(m: int, n: int, seed: int = 0) -> np.ndarray:
    """i.i.d. N(0,1) entries."""
    return _rng(seed).standard_normal((m, n), dtype=np.float32)


def lowrank_outliers(m: int, n: int, seed: int = 0, rank: int = 64, noise: float = 0.1,
                     outlier_frac: float = 1e-3, outlier_scale: float = 20.0) -> np.ndarray:
    """Rank-`rank` Gaussian component of unit entry variance plus N(0, noise^2)
    noise; a Bernoulli(outlier_frac) mask of entries is replaced by
    outlier_scale * Student-t(nu=3) samples."""
    g = _rng(seed)
    u = g.standard_normal((m, rank), dtype=np.float32)
    v = g.standard_normal((n, rank), dtype=np.float32)
    x = (u @ v.T) / np.float32(np.sqrt(rank))
    x += np.float32(noise) * g.standard_normal((m, n), dtype=np.float32)
    mask = g.random((m, n), dtype=np.float32) < np.float32(outlier_frac)
    t = g.standard_t(3.0, size=int(mask.sum())).astype(np.float32)
    x[mask] = np.float32(outlier_scale) * t
    return np.ascontiguousarray(x, dtype=np.float32)


def row_lognormal(m: int, n: int, seed: int = 0) -> np.ndarray:
    """N(0,1) entries, each row multiplied by an exp(N(0,1)) magnitude."""
    g = _rng(seed)
    x = g.standard_normal((m, n), dtype=np.float32)
    x *= np.exp(g.standard_normal((m, 1), dtype=np.float32))
    return np.ascontiguousarray(x, dtype=np.float32)


def gradient_like(m: int, n: int, seed: int = 0, rank: int = 32,
                  outlier_frac: float = 5e-4, outlier_scale: float = 20.0) -> np.ndarray:
    """N(0,1) entries plus a rank-`rank` Gaussian term of unit entry variance;
    a Bernoulli(outlier_frac) mask of entries is multiplied by outlier_scale."""
    g = _rng(seed)
    x = g.standard_normal((m, n), dtype=np.float32)
    u = g.standard_normal((m, rank), dtype=np.float32)
    v = g.standard_normal((n, rank), dtype=np.float32)
    x += (u @ v.T) / np.float32(np.sqrt(rank))
    mask = g.random((m, n), dtype=np.float32) < np.float32(outlier_frac)
    x[mask] *= np.float32(outlier_scale)
    return np.ascontiguousarray(x, dtype=np.float32)


# --- the five configurations ---------------------------------------------------
ROLES_3B = (("Wq", 3072, 3072), ("Wk", 3072, 3072), ("Wv", 3072, 3072), ("Wo", 3072, 3072),
            ("Wgate", 3072, 8192), ("Wup", 3072, 8192), ("Wdown", 8192, 3072))


def config1() -> np.ndarray:
    return gaussian(256, 512, seed=0)


def config2() -> np.ndarray:
    return lowrank_outliers(2048, 2048, seed=0)


def config3():
    return row_lognormal(2048, 8192, seed=0), row_lognormal(8192, 2048, seed=1)


def stack_3b_shapes(blocks: int = 4):
    """(name, m, n, seed) of the decoder-stack batch: hidden 3072, FFN 8192 gated."""
    out = []
    for b in range(blocks):
        for r, (name, m, n) in enumerate(ROLES_3B):
            out.append((f"block{b}.{name}", m, n, 1000 * b + r))
    return out


def stack_3b(blocks: int = 4, scale_down: int = 1):
    """The 7 * blocks matrices of the decoder-stack batch.  scale_down divides
    every dimension (for small parity cases); it must keep them multiples of 128."""
    mats = []
    for name, m, n, seed in stack_3b_shapes(blocks):
        mats.append(gradient_like(m // scale_down, n // scale_down, seed=seed))
    return mats


def gqa_stack_shapes(d: int, d_ff: int, kv: int = 1024, blocks: int = 4, fused: bool = False):
    """(name, m, n) of the projections of `blocks` decoder blocks with hidden size d, gated FFN
    width d_ff and grouped-query attention whose key / value projections are kv wide (the
    paper's timing shapes: Section 4.3, d = 4096 / 6144, d_ff = 11008 / 13824, 8 KV heads of
    128).  Weights are stored (out, in).  fused: one qkv and one gate_up matrix per block."""
    if fused:
        roles = (("Wqkv", d + 2 * kv, d), ("Wo", d, d), ("Wgate_up", 2 * d_ff, d), ("Wdown", d, d_ff))
    else:
        roles = (("Wq", d, d), ("Wk", kv, d), ("Wv", kv, d), ("Wo", d, d), ("Wgate", d_ff, d), ("Wup", d_ff, d),
                 ("Wdown", d, d_ff))
    return [(f"block{b}.{name}", m, n) for b in range(blocks) for name, m, n in roles]


def sweep_square(size: int) -> np.ndarray:
    return gaussian(size, size, seed=1)
