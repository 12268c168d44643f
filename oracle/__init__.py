"""ctypes front end of the CPU oracle (test infrastructure, not product code).

The oracle is ``nvfp4_oracle.cpp`` beside this file: a plain scalar C++
restatement of the NVFP4 Root Newton-Schulz step.  Only tests, the smoke check
and the benchmark's CPU-baseline leg may import this package; the CUDA library
and its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nvfp4_oracle.cpp")
_LIB = os.path.join(_HERE, "libnvfp4_oracle.so")
_lib = None

_u8p = C.POINTER(C.c_uint8)
_f32p = C.POINTER(C.c_float)
_u16p = C.POINTER(C.c_uint16)
_u32p = C.POINTER(C.c_uint32)


class OrcParams(C.Structure):
    _fields_ = [("a", C.c_float), ("b", C.c_float), ("c", C.c_float),
                ("clip_quantile", C.c_float), ("eps", C.c_float),
                ("quantize", C.c_int32), ("exact_scales", C.c_int32),
                ("rht", C.c_int32), ("four_six", C.c_int32), ("seed", C.c_uint64),
                ("store_bf16", C.c_int32)]


class OrcTrace(C.Structure):
    _fields_ = [("iter", C.c_int32),
                ("tau", _f32p), ("nu", _f32p), ("X0", _f32p), ("amax_in", _f32p), ("X_in", _f32p),
                ("qX_codes", _u8p), ("qX_scales", _u8p), ("qXt_codes", _u8p), ("qXt_scales", _u8p),
                ("sg_X", _f32p), ("A", _f32p),
                ("qA_codes", _u8p), ("qA_scales", _u8p), ("sg_A", _f32p),
                ("S", _f32p), ("B", _f32p),
                ("qB_codes", _u8p), ("qB_scales", _u8p), ("sg_B", _f32p),
                ("X_out", _f32p)]


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved); returns the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
           _SRC, "-o", _LIB]
    subprocess.run(cmd, check=True)
    return _LIB


class AdamWParams(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("step", C.c_int32), ("sr", C.c_int32), ("seed", C.c_uint64)]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_e2m1_encode.argtypes = [C.c_float]; L.orc_e2m1_encode.restype = C.c_uint8
        L.orc_e2m1_decode.argtypes = [C.c_uint8]; L.orc_e2m1_decode.restype = C.c_float
        L.orc_ue4m3_encode.argtypes = [C.c_float]; L.orc_ue4m3_encode.restype = C.c_uint8
        L.orc_ue4m3_decode.argtypes = [C.c_uint8]; L.orc_ue4m3_decode.restype = C.c_float
        L.orc_amax.argtypes = [_f32p, C.c_int64]; L.orc_amax.restype = C.c_float
        L.orc_tensor_scale_exact.argtypes = [C.c_float]; L.orc_tensor_scale_exact.restype = C.c_float
        L.orc_tensor_scale_predicted.argtypes = [C.c_float]; L.orc_tensor_scale_predicted.restype = C.c_float
        L.orc_quantile_rank.argtypes = [C.c_int64, C.c_float]; L.orc_quantile_rank.restype = C.c_int64
        L.orc_quantize.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_float, _u8p, _u8p]
        L.orc_quantize.restype = None
        L.orc_quantize_opts.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_float, _u8p, _u8p, C.c_int, C.c_uint16, C.c_int]
        L.orc_quantize_opts.restype = None
        L.orc_hadamard16.argtypes = [_f32p, C.c_uint16, _f32p]; L.orc_hadamard16.restype = None
        L.orc_rht_mask.argtypes = [C.c_uint64, C.c_uint64]; L.orc_rht_mask.restype = C.c_uint16
        L.orc_bf16_round.argtypes = [C.c_float]; L.orc_bf16_round.restype = C.c_float
        L.orc_momentum_encode.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_int, C.c_uint64, _u8p, _u16p]
        L.orc_momentum_encode.restype = None
        L.orc_momentum_decode.argtypes = [_u8p, _u16p, C.c_int64, C.c_int64, _f32p]
        L.orc_momentum_decode.restype = None
        L.orc_momentum_update.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_float, C.c_float, C.c_int, C.c_uint64,
                                          _u8p, _u16p, _f32p, _u32p]
        L.orc_momentum_update.restype = None
        L.orc_v_encode.argtypes = [_f32p, C.c_int64, _u8p, _u16p, _u16p]; L.orc_v_encode.restype = None
        L.orc_v_decode.argtypes = [_u8p, _u16p, _u16p, C.c_int64, _f32p]; L.orc_v_decode.restype = None
        L.orc_adamw_update.argtypes = [_u16p, _u16p, C.c_int64, _u8p, _u16p, _u8p, _u16p, _u16p,
                                       C.POINTER(AdamWParams), _f32p, _f32p]
        L.orc_adamw_update.restype = None
        L.orc_splitmix64_at.argtypes = [C.c_uint64, C.c_uint64]; L.orc_splitmix64_at.restype = C.c_uint64
        L.orc_dequantize.argtypes = [_u8p, _u8p, C.c_float, C.c_int64, C.c_int64, _f32p]
        L.orc_dequantize.restype = None
        L.orc_gemm_nt_q.argtypes = [_u8p, _u8p, C.c_float, _u8p, _u8p, C.c_float,
                                    C.c_int64, C.c_int64, C.c_int64, _f32p, C.c_int]
        L.orc_gemm_nt_q.restype = None
        L.orc_clip_threshold.argtypes = [_f32p, C.c_int64, C.c_float]
        L.orc_clip_threshold.restype = C.c_float
        L.orc_root_coeffs.argtypes = [C.c_int64, C.c_int64, C.c_int, _f32p]
        L.orc_root_coeffs.restype = None
        L.orc_root_ns.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_int, C.POINTER(OrcParams),
                                  _f32p, C.POINTER(OrcTrace)]
        L.orc_root_ns.restype = C.c_int
        L.orc_root_param_update.argtypes = [_u16p, _f32p, C.c_int64, C.c_float, C.c_float, C.c_float]
        L.orc_root_param_update.restype = None
        L.orc_sr_e2m1x4.argtypes = [_f32p, C.c_uint32]; L.orc_sr_e2m1x4.restype = C.c_uint16
        L.orc_ns_iteration.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_float, C.c_float,
                                       C.POINTER(OrcParams), _f32p, _f32p, _f32p, C.POINTER(OrcTrace)]
        L.orc_ns_iteration.restype = C.c_int
        _lib = L
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _u8(a):
    a = np.ascontiguousarray(a, dtype=np.uint8)
    return a, a.ctypes.data_as(_u8p)


# --- codecs -----------------------------------------------------------------
def e2m1_encode(y: float) -> int:
    return int(lib().orc_e2m1_encode(float(np.float32(y))))


def e2m1_decode(nib: int) -> float:
    return float(lib().orc_e2m1_decode(int(nib)))


def ue4m3_encode(t: float) -> int:
    return int(lib().orc_ue4m3_encode(float(np.float32(t))))


def ue4m3_decode(b: int) -> float:
    return float(lib().orc_ue4m3_decode(int(b)))


def tensor_scale_exact(amax: float) -> float:
    return float(lib().orc_tensor_scale_exact(float(np.float32(amax))))


def tensor_scale_predicted(bound: float) -> float:
    return float(lib().orc_tensor_scale_predicted(float(np.float32(bound))))


def quantile_rank(n: int, q: float) -> int:
    return int(lib().orc_quantile_rank(int(n), float(np.float32(q))))


# --- quantiser ----------------------------------------------------------------
def quantize(x, s_g=None, rht=False, mask=0, four_six=False):
    """Q_1x16 of a 2-D FP32 array.  s_g None: exact rule amax/2688 (4 amax/2688 with rht).
    rht: every 16-block is first multiplied by the random Hadamard matrix of `mask`;
    four_six: adaptive 4/6 block scaling.

    Returns (codes[rows, cols/2] u8, scales[rows, cols/16] u8, s_g)."""
    x, xp = _f32(x)
    rows, cols = x.shape
    assert cols % 16 == 0
    if s_g is None:
        amax = float(lib().orc_amax(xp, x.size))
        s_g = tensor_scale_exact(float(np.float32(4.0) * np.float32(amax)) if rht else amax)
    codes = np.empty((rows, cols // 2), np.uint8)
    scales = np.empty((rows, cols // 16), np.uint8)
    lib().orc_quantize_opts(xp, rows, cols, float(np.float32(s_g)), codes.ctypes.data_as(_u8p),
                            scales.ctypes.data_as(_u8p), int(bool(rht)), int(mask), int(bool(four_six)))
    return codes, scales, float(np.float32(s_g))


def hadamard16(x, mask=0):
    """x diag(r) H_16 / 4 for one block of 16 (bit i of mask set: r_i = -1)."""
    x, xp = _f32(x)
    y = np.empty(16, np.float32)
    lib().orc_hadamard16(xp, int(mask), y.ctypes.data_as(_f32p))
    return y


def rht_mask(seed, idx):
    return int(lib().orc_rht_mask(int(seed), int(idx)))


def bf16_round(x):
    """FP32 -> nearest BF16 (ties to even), as FP32; scalar or array."""
    f = np.vectorize(lambda v: lib().orc_bf16_round(float(v)), otypes=[np.float32])
    return f(np.asarray(x, np.float32))


def splitmix64_at(seed, idx):
    """Output number idx (from 0) of the splitmix64 generator seeded with `seed`."""
    return int(lib().orc_splitmix64_at(int(seed), int(idx)))


def root_param_update(W_bits, O, lr, weight_decay=0.0, scale=1.0):
    """Root's parameter update on BF16 weights (bit patterns, uint16): returns the new bit patterns."""
    W = np.ascontiguousarray(W_bits, dtype=np.uint16).copy()
    O_, op = _f32(O)
    assert W.shape == O_.shape
    lib().orc_root_param_update(W.ctypes.data_as(_u16p), op, W.size, float(np.float32(lr)),
                                float(np.float32(weight_decay)), float(np.float32(scale)))
    return W


def sr_e2m1x4(y4, word: int) -> int:
    """Four values rounded stochastically with one 32-bit random word; four nibbles, element 0 lowest."""
    y, yp = _f32(np.asarray(y4, np.float32).reshape(4))
    return int(lib().orc_sr_e2m1x4(yp, int(word) & 0xFFFFFFFF))


def momentum_encode(M, sr=False, seed=0):
    """First-moment state of an FP32 matrix: (codes u8 rows x cols/2, scales u16 rows x cols/16)."""
    M, mp = _f32(M)
    rows, cols = M.shape
    codes = np.empty((rows, cols // 2), np.uint8)
    scales = np.empty((rows, cols // 16), np.uint16)
    lib().orc_momentum_encode(mp, rows, cols, int(bool(sr)), int(seed), codes.ctypes.data_as(_u8p),
                              scales.ctypes.data_as(_u16p))
    return codes, scales


def momentum_decode(codes, scales):
    codes, cp = _u8(codes)
    scales = np.ascontiguousarray(scales, np.uint16)
    rows, cols = codes.shape[0], codes.shape[1] * 2
    out = np.empty((rows, cols), np.float32)
    lib().orc_momentum_decode(cp, scales.ctypes.data_as(_u16p), rows, cols, out.ctypes.data_as(_f32p))
    return out


def momentum_update(G, codes, scales, mu, g_scale=1.0, sr=False, seed=0, want_hist=True):
    """One step on a stored state; returns (M_t, new codes, new scales, histogram or None)."""
    G, gp = _f32(G)
    rows, cols = G.shape
    codes = np.array(codes, np.uint8, copy=True)
    scales = np.array(scales, np.uint16, copy=True)
    M = np.empty((rows, cols), np.float32)
    hist = np.zeros(8192, np.uint32) if want_hist else None
    lib().orc_momentum_update(gp, rows, cols, float(np.float32(mu)), float(np.float32(g_scale)), int(bool(sr)),
                              int(seed), codes.ctypes.data_as(_u8p), scales.ctypes.data_as(_u16p),
                              M.ctypes.data_as(_f32p),
                              hist.ctypes.data_as(_u32p) if want_hist else None)
    return M, codes, scales, hist


def bf16_bits(x):
    """FP32 array -> BF16 bit patterns (uint16), round to nearest even."""
    r = bf16_round(np.asarray(x, np.float32))
    return (np.ascontiguousarray(r).view(np.uint32) >> 16).astype(np.uint16)


def bf16_to_f32(bits):
    return (np.asarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)


def v_encode(v):
    """Second-moment state of a flat FP32 array (length a multiple of 256):
    (codes u8 n/2, scales u16 n/16, means u16 n/256)."""
    v, vp = _f32(np.asarray(v, np.float32).ravel())
    n = v.size
    codes = np.empty(n // 2, np.uint8); scales = np.empty(n // 16, np.uint16); means = np.empty(n // 256, np.uint16)
    lib().orc_v_encode(vp, n, codes.ctypes.data_as(_u8p), scales.ctypes.data_as(_u16p), means.ctypes.data_as(_u16p))
    return codes, scales, means


def v_decode(codes, scales, means):
    codes = np.ascontiguousarray(codes, np.uint8); scales = np.ascontiguousarray(scales, np.uint16)
    means = np.ascontiguousarray(means, np.uint16)
    n = codes.size * 2
    out = np.empty(n, np.float32)
    lib().orc_v_decode(codes.ctypes.data_as(_u8p), scales.ctypes.data_as(_u16p), means.ctypes.data_as(_u16p), n,
                       out.ctypes.data_as(_f32p))
    return out


def adamw_update(W_bits, G_bits, state, lr, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, step=1, sr=False,
                 seed=0):
    """One packed AdamW step.  state = (m_codes, m_scales, v_codes, v_scales, v_means) or None for
    zeros.  Returns (W_bits, new state, m FP32, v FP32); inputs are not modified."""
    W = np.array(W_bits, np.uint16, copy=True).ravel()
    G = np.ascontiguousarray(G_bits, np.uint16).ravel()
    n = W.size
    if state is None:
        state = (np.zeros(n // 2, np.uint8), np.zeros(n // 16, np.uint16), np.zeros(n // 2, np.uint8),
                 np.zeros(n // 16, np.uint16), np.zeros(n // 256, np.uint16))
    mc, ms, vc, vs, vm = [np.array(a, copy=True) for a in state]
    m = np.empty(n, np.float32); v = np.empty(n, np.float32)
    prm = AdamWParams(lr, beta1, beta2, eps, weight_decay, step, int(bool(sr)), seed)
    lib().orc_adamw_update(W.ctypes.data_as(_u16p), G.ctypes.data_as(_u16p), n, mc.ctypes.data_as(_u8p),
                           ms.ctypes.data_as(_u16p), vc.ctypes.data_as(_u8p), vs.ctypes.data_as(_u16p),
                           vm.ctypes.data_as(_u16p), C.byref(prm), m.ctypes.data_as(_f32p), v.ctypes.data_as(_f32p))
    return W, (mc, ms, vc, vs, vm), m, v


def dequantize(codes, scales, s_g):
    codes, cp = _u8(codes)
    scales, sp = _u8(scales)
    rows, cols = codes.shape[0], codes.shape[1] * 2
    out = np.empty((rows, cols), np.float32)
    lib().orc_dequantize(cp, sp, float(np.float32(s_g)), rows, cols, out.ctypes.data_as(_f32p))
    return out


def gemm_nt_q(a, b=None):
    """FP32(deq(a) @ deq(b).T) with FP64 sums; a, b = (codes, scales, s_g).
    b None: symmetric product a a^T (upper triangle computed, mirrored)."""
    ac, acp = _u8(a[0]); as_, asp = _u8(a[1])
    M, K = ac.shape[0], ac.shape[1] * 2
    if b is None:
        out = np.empty((M, M), np.float32)
        lib().orc_gemm_nt_q(acp, asp, float(a[2]), acp, asp, float(a[2]), M, M, K,
                            out.ctypes.data_as(_f32p), 1)
        return out
    bc, bcp = _u8(b[0]); bs, bsp = _u8(b[1])
    N = bc.shape[0]
    assert bc.shape[1] * 2 == K
    out = np.empty((M, N), np.float32)
    lib().orc_gemm_nt_q(acp, asp, float(a[2]), bcp, bsp, float(b[2]), M, N, K,
                        out.ctypes.data_as(_f32p), 0)
    return out


# --- clip, coefficients, the whole step ---------------------------------------
def clip_threshold(g, q=0.99) -> float:
    g, gp = _f32(g)
    return float(lib().orc_clip_threshold(gp, g.size, float(np.float32(q))))


def root_coeffs(m, n, steps=5):
    abc = (C.c_float * 3)()
    lib().orc_root_coeffs(int(m), int(n), int(steps), abc)
    return float(abc[0]), float(abc[1]), float(abc[2])


def root_ns(G, steps=5, abc=None, clip_quantile=0.99, eps=1e-7, quantize=True,
            exact_scales=False, trace_iter=None, rht=False, four_six=False, seed=0, store_bf16=False):
    """The Root Newton-Schulz step on one m x n FP32 matrix.

    Returns out (m x n FP32), or (out, trace dict) when trace_iter is given; the
    trace holds the intermediates of that iteration in the work orientation
    (s x l, s = min(m, n))."""
    G, gp = _f32(G)
    m, n = G.shape
    s, l = min(m, n), max(m, n)
    p = OrcParams()
    if abc is None:
        p.a = p.b = p.c = float("nan")
    else:
        p.a, p.b, p.c = [float(np.float32(v)) for v in abc]
    p.clip_quantile = float(np.float32(clip_quantile))
    p.eps = float(np.float32(eps))
    p.quantize = 1 if quantize else 0
    p.exact_scales = 1 if exact_scales else 0
    p.rht = 1 if rht else 0
    p.four_six = 1 if four_six else 0
    p.seed = int(seed)
    p.store_bf16 = 1 if store_bf16 else 0
    out = np.empty((m, n), np.float32)
    if trace_iter is None:
        rc = lib().orc_root_ns(gp, m, n, int(steps), C.byref(p), out.ctypes.data_as(_f32p), None)
        if rc:
            raise ValueError(f"orc_root_ns failed with code {rc}")
        return out
    t, bufs = _make_trace(s, l, quantize)
    t.iter = int(trace_iter)
    rc = lib().orc_root_ns(gp, m, n, int(steps), C.byref(p), out.ctypes.data_as(_f32p), C.byref(t))
    if rc:
        raise ValueError(f"orc_root_ns failed with code {rc}")
    return out, _finish_trace(bufs)


def _make_trace(s, l, quantize=True):
    t = OrcTrace()
    bufs = {}

    def f(name, shape):
        bufs[name] = np.zeros(shape, np.float32)
        setattr(t, name, bufs[name].ctypes.data_as(_f32p))

    def u(name, shape):
        bufs[name] = np.zeros(shape, np.uint8)
        setattr(t, name, bufs[name].ctypes.data_as(_u8p))

    for name in ("tau", "nu", "amax_in", "sg_X", "sg_A", "sg_B"):
        f(name, (1,))
    for name in ("X0", "X_in", "X_out"):
        f(name, (s, l))
    for name in ("A", "S", "B"):
        f(name, (s, s))
    if quantize:
        u("qX_codes", (s, l // 2)); u("qX_scales", (s, l // 16))
        u("qXt_codes", (l, s // 2)); u("qXt_scales", (l, s // 16))
        u("qA_codes", (s, s // 2)); u("qA_scales", (s, s // 16))
        u("qB_codes", (s, s // 2)); u("qB_scales", (s, s // 16))
    return t, bufs


def _finish_trace(bufs):
    for name in ("tau", "nu", "amax_in", "sg_X", "sg_A", "sg_B"):
        bufs[name] = float(bufs[name][0])
    return bufs


def ns_iteration(X, k, amax_X, sg_X, abc=None, last=False, rht=False, four_six=False, seed=0):
    """One quantised Newton-Schulz iteration (index k) from a given state: X is s x l FP32 in the
    work orientation (s <= l), amax_X = max|X|, sg_X the tensor scale of its operand copies.
    Returns (X_next, amax_next, sg_next, trace dict)."""
    X, xp = _f32(X)
    s, l = X.shape
    p = OrcParams()
    if abc is None:
        p.a = p.b = p.c = float("nan")
    else:
        p.a, p.b, p.c = [float(np.float32(v)) for v in abc]
    p.clip_quantile = 0.0
    p.eps = 0.0
    p.quantize = 1
    p.exact_scales = 0
    p.rht = 1 if rht else 0
    p.four_six = 1 if four_six else 0
    p.seed = int(seed)
    p.store_bf16 = 0
    t, bufs = _make_trace(s, l)
    t.iter = int(k)
    out = np.empty((s, l), np.float32)
    am = np.zeros(1, np.float32); sg = np.zeros(1, np.float32)
    rc = lib().orc_ns_iteration(xp, s, l, int(k), 1 if last else 0, float(np.float32(amax_X)), float(np.float32(sg_X)),
                                C.byref(p), out.ctypes.data_as(_f32p), am.ctypes.data_as(_f32p),
                                sg.ctypes.data_as(_f32p), C.byref(t))
    if rc:
        raise ValueError(f"orc_ns_iteration failed with code {rc}")
    return out, float(am[0]), float(sg[0]), _finish_trace(bufs)
