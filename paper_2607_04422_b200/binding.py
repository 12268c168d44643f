"""ctypes binding of libfp4root.so: argument marshalling only.

Functions carry the names of the C ABI (include/fp4root.h).  Tensors are torch CUDA
tensors used purely as device memory; streams are torch streams.  Every step of the
path runs in the library's kernels; if the library is missing the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.environ.get("FP4ROOT_LIB") or os.path.join(_HERE, "libfp4root.so")
_lib = None

FP4_FLAG_KEEP_OPERANDS = 1
FP4_FLAG_RHT = 2
FP4_FLAG_FOUR_SIX = 4
FP4_FLAG_STORE_BF16 = 8
FP4_FLAG_NO_OUT = 16
FP4_FLAG_OVERLAP_GROUPS = 32
FP4_MOM_FLAG_SR = 1
STATUS_NAMES = {0: "FP4_OK", 1: "FP4_ERR_INVALID_ARG", 2: "FP4_ERR_SHAPE", 3: "FP4_ERR_ALIGNMENT",
                4: "FP4_ERR_WORKSPACE", 5: "FP4_ERR_ARCH", 6: "FP4_ERR_CUDA", 7: "FP4_ERR_DEVICE_TIMEOUT",
                8: "FP4_ERR_UNIMPLEMENTED", 9: "FP4_ERR_STATIC_LIMIT"}
FP4_STATIC_SCRATCH_BYTES = 16 << 20

EXPORTS = ("fp4_status_string", "fp4_scale_bytes", "fp4_quantize", "fp4_root_coeffs",
           "fp4_root_ns_workspace_bytes", "fp4_root_ns", "fp4_root_ns_batched_workspace_bytes",
           "fp4_root_ns_batched", "fp4_last_device_status", "fp4_root_ns_workspace_layout", "fp4_gemm_nt",
           "fp4_gemm_nt_resident",
           "fp4_profile_enable", "fp4_profile_collect", "fp4_kernel_launches", "fp4_root_ns_static",
           "fp4_selftest_bounded_wait")
PROF_CLASSES = ("clip", "stats", "prep", "G1", "G2", "G3", "transpose", "quantize", "momentum", "adamw")


class Fp4Error(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        super().__init__(f"{where}: {STATUS_NAMES.get(self.code, self.code)} ({fp4_status_string(self.code)})")


class NsParams(C.Structure):
    """fp4_ns_params"""
    _fields_ = [("a", C.c_float), ("b", C.c_float), ("c", C.c_float), ("clip_quantile", C.c_float),
                ("eps", C.c_float), ("flags", C.c_uint32), ("max_group", C.c_uint32), ("seed", C.c_uint64),
                ("top_hist", C.POINTER(C.c_void_p)), ("weights", C.POINTER(C.c_void_p)),
                ("lr", C.c_float), ("weight_decay", C.c_float), ("update_scale", C.c_float)]

    @classmethod
    def make(cls, abc=None, clip_quantile=0.99, eps=1e-7, flags=0, max_group=0, seed=0, top_hist=None,
             weights=None, lr=0.0, weight_decay=0.0, update_scale=1.0):
        p = cls()
        if abc is None:
            p.a = p.b = p.c = float("nan")
        else:
            p.a, p.b, p.c = [float(v) for v in abc]
        p.clip_quantile, p.eps, p.flags = float(clip_quantile), float(eps), int(flags)
        p.max_group = int(max_group)
        p.seed = int(seed)
        if top_hist is not None:
            # one entry per matrix of the call: a tensor of 8192 int32 counters, or None
            arr = (C.c_void_p * len(top_hist))(*[h.data_ptr() if h is not None else None for h in top_hist])
            p._top_hist_keepalive = arr
            p.top_hist = C.cast(arr, C.POINTER(C.c_void_p))
        if weights is not None:
            # one entry per matrix of the call: a BF16 tensor of the matrix's shape, or None
            arr = (C.c_void_p * len(weights))(*[w.data_ptr() if w is not None else None for w in weights])
            p._weights_keepalive = arr
            p.weights = C.cast(arr, C.POINTER(C.c_void_p))
        p.lr, p.weight_decay, p.update_scale = float(lr), float(weight_decay), float(update_scale)
        return p


class MomentumParams(C.Structure):
    """fp4_momentum_params of include/fp4root.h."""
    _fields_ = [("mu", C.c_float), ("g_scale", C.c_float), ("flags", C.c_uint32), ("reserved", C.c_uint32),
                ("seed", C.c_uint64)]


class AdamwParams(C.Structure):
    """fp4_adamw_params of include/fp4root.h."""
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("step", C.c_int32), ("flags", C.c_uint32), ("reserved", C.c_uint32),
                ("seed", C.c_uint64)]


class WsLayout(C.Structure):
    """fp4_ws_layout"""
    _fields_ = [("header", C.c_size_t), ("scalars", C.c_size_t), ("X", C.c_size_t), ("A", C.c_size_t),
                ("qX_codes", C.c_size_t), ("qX_scales", C.c_size_t),
                ("qXt_codes", C.c_size_t * 2), ("qXt_scales", C.c_size_t * 2),
                ("qA_codes", C.c_size_t), ("qA_scales", C.c_size_t),
                ("qB_codes", C.c_size_t), ("qB_scales", C.c_size_t),
                ("idx_tau", C.c_int32), ("idx_nu", C.c_int32), ("idx_inv", C.c_int32),
                ("idx_amax_X0", C.c_int32), ("idx_amax_A0", C.c_int32),
                ("idx_sg_X0", C.c_int32), ("idx_sg_A0", C.c_int32), ("idx_sg_B0", C.c_int32),
                ("total", C.c_size_t), ("Xh", C.c_size_t)]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libfp4root.so (built in-tree by build.py).  Raises if it is missing:
    there is no fallback implementation."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2607_04422_b200.build` "
                           "(nvcc, sm_100a); this package has no CPU or PyTorch fallback")
    L = C.CDLL(_LIB_PATH)
    vp, i64, u32, sz = C.c_void_p, C.c_int64, C.c_uint32, C.c_size_t
    L.fp4_status_string.argtypes = [C.c_int]; L.fp4_status_string.restype = C.c_char_p
    L.fp4_scale_bytes.argtypes = [i64, i64]; L.fp4_scale_bytes.restype = sz
    L.fp4_quantize.argtypes = [vp, i64, i64, vp, vp, vp, u32, vp]; L.fp4_quantize.restype = C.c_int
    L.fp4_root_coeffs.argtypes = [i64, i64, C.c_int, C.POINTER(C.c_float)]; L.fp4_root_coeffs.restype = C.c_int
    L.fp4_root_ns_workspace_bytes.argtypes = [i64, i64, C.c_int, u32]; L.fp4_root_ns_workspace_bytes.restype = sz
    L.fp4_root_ns.argtypes = [vp, vp, i64, i64, C.c_int, C.POINTER(NsParams), vp, sz, vp]
    L.fp4_root_ns.restype = C.c_int
    L.fp4_root_ns_batched_workspace_bytes.argtypes = [C.c_int, C.POINTER(i64), C.POINTER(i64), C.c_int, u32]
    L.fp4_root_ns_batched_workspace_bytes.restype = sz
    L.fp4_root_ns_batched.argtypes = [C.c_int, C.POINTER(vp), C.POINTER(vp), C.POINTER(i64), C.POINTER(i64),
                                      C.c_int, C.POINTER(NsParams), vp, sz, vp]
    L.fp4_root_ns_batched.restype = C.c_int
    L.fp4_last_device_status.argtypes = [vp, vp]; L.fp4_last_device_status.restype = C.c_int
    L.fp4_root_ns_workspace_layout.argtypes = [i64, i64, C.c_int, u32, C.POINTER(WsLayout)]
    L.fp4_root_ns_workspace_layout.restype = C.c_int
    L.fp4_gemm_nt.argtypes = [vp, vp, C.c_float, vp, vp, C.c_float, i64, i64, i64, vp, vp, vp]
    L.fp4_gemm_nt.restype = C.c_int
    L.fp4_gemm_nt_resident.argtypes = L.fp4_gemm_nt.argtypes
    L.fp4_gemm_nt_resident.restype = C.c_int
    L.fp4_root_ns_static.argtypes = [vp, vp, i64, i64, C.c_int, C.POINTER(NsParams), vp, vp]
    L.fp4_root_ns_static.restype = C.c_int
    L.fp4_profile_enable.argtypes = [C.c_int]; L.fp4_profile_enable.restype = None
    L.fp4_profile_collect.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_int)]
    L.fp4_profile_collect.restype = C.c_int
    L.fp4_kernel_launches.argtypes = []; L.fp4_kernel_launches.restype = C.c_uint64
    L.fp4_momentum_update.argtypes = [vp, i64, i64, vp, vp, vp, vp, C.POINTER(MomentumParams), vp]
    L.fp4_momentum_update.restype = C.c_int
    L.fp4_adamw_update.argtypes = [vp, vp, i64, vp, vp, vp, vp, vp, C.POINTER(AdamwParams), vp]
    L.fp4_adamw_update.restype = C.c_int
    L.fp4_momentum_decode.argtypes = [vp, vp, i64, i64, vp, vp]; L.fp4_momentum_decode.restype = C.c_int
    L.fp4_selftest_bounded_wait.argtypes = [vp, u32, vp]; L.fp4_selftest_bounded_wait.restype = C.c_int
    _lib = L
    return L


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _check(rc: int, where: str):
    if rc != 0:
        raise Fp4Error(rc, where)


def fp4_status_string(code: int) -> str:
    return load_library().fp4_status_string(int(code)).decode()


def fp4_scale_bytes(rows: int, cols: int) -> int:
    return int(load_library().fp4_scale_bytes(rows, cols))


def fp4_root_coeffs(m: int, n: int, steps: int = 5):
    abc = (C.c_float * 3)()
    _check(load_library().fp4_root_coeffs(m, n, steps, abc), "fp4_root_coeffs")
    return float(abc[0]), float(abc[1]), float(abc[2])


def fp4_quantize(x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, tensor_scale: torch.Tensor,
                 flags: int = 0, stream=None) -> None:
    rows, cols = x.shape
    _check(load_library().fp4_quantize(x.data_ptr(), rows, cols, codes.data_ptr(), scales.data_ptr(),
                                       tensor_scale.data_ptr(), flags, _stream(stream)), "fp4_quantize")


def fp4_momentum_update(G: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, M_out: torch.Tensor | None,
                        hist: torch.Tensor | None, mu: float, g_scale: float = 1.0, flags: int = 0, seed: int = 0,
                        stream=None) -> None:
    """One momentum step on the 5-bit state (codes uint8 rows x cols/2, scales int16/uint16 rows x cols/16),
    in place; M_out (FP32) and hist (8192 int32 counters, added to) are optional."""
    rows, cols = G.shape
    prm = MomentumParams(mu, g_scale, flags, 0, seed)
    _check(load_library().fp4_momentum_update(G.data_ptr(), rows, cols, codes.data_ptr(), scales.data_ptr(),
                                              M_out.data_ptr() if M_out is not None else None,
                                              hist.data_ptr() if hist is not None else None, C.byref(prm),
                                              _stream(stream)), "fp4_momentum_update")


def fp4_adamw_update(W: torch.Tensor, G: torch.Tensor, m_codes: torch.Tensor, m_scales: torch.Tensor,
                     v_codes: torch.Tensor, v_scales: torch.Tensor, v_means: torch.Tensor, lr: float,
                     beta1: float = 0.9, beta2: float = 0.95, eps: float = 1e-8, weight_decay: float = 0.1,
                     step: int = 1, flags: int = 0, seed: int = 0, stream=None) -> None:
    """One packed AdamW step in place on BF16 weights W with BF16 gradients G (flat, a multiple of
    256 elements) and both moments in their NVFP4 states."""
    prm = AdamwParams(lr, beta1, beta2, eps, weight_decay, step, flags, 0, seed)
    _check(load_library().fp4_adamw_update(W.data_ptr(), G.data_ptr(), W.numel(), m_codes.data_ptr(),
                                           m_scales.data_ptr(), v_codes.data_ptr(), v_scales.data_ptr(),
                                           v_means.data_ptr(), C.byref(prm), _stream(stream)), "fp4_adamw_update")


def fp4_momentum_decode(codes: torch.Tensor, scales: torch.Tensor, M_out: torch.Tensor, stream=None) -> None:
    rows, cols = M_out.shape
    _check(load_library().fp4_momentum_decode(codes.data_ptr(), scales.data_ptr(), rows, cols, M_out.data_ptr(),
                                              _stream(stream)), "fp4_momentum_decode")


def fp4_root_ns_workspace_bytes(m: int, n: int, steps: int = 5, flags: int = 0) -> int:
    return int(load_library().fp4_root_ns_workspace_bytes(m, n, steps, flags))


def fp4_root_ns_workspace_layout(m: int, n: int, steps: int = 5, flags: int = 0) -> WsLayout:
    lay = WsLayout()
    _check(load_library().fp4_root_ns_workspace_layout(m, n, steps, flags, C.byref(lay)),
           "fp4_root_ns_workspace_layout")
    return lay


def fp4_root_ns(G: torch.Tensor, out: torch.Tensor, steps: int, params: NsParams | None, ws: torch.Tensor,
                stream=None) -> None:
    m, n = G.shape
    p = C.byref(params) if params is not None else None
    _check(load_library().fp4_root_ns(G.data_ptr(), out.data_ptr(), m, n, steps, p, ws.data_ptr(),
                                      ws.numel() * ws.element_size(), _stream(stream)), "fp4_root_ns")


def fp4_root_ns_static(G: torch.Tensor, out: torch.Tensor, steps: int, params: NsParams | None = None,
                       device_status: torch.Tensor | None = None, stream=None) -> None:
    """fp4_root_ns for callers that cannot allocate a workspace: the library's own 16 MiB
    static device array is the scratch.  Shapes that need more raise FP4_ERR_STATIC_LIMIT.
    Calls that could overlap on the GPU must be ordered by the caller."""
    m, n = G.shape
    p = C.byref(params) if params is not None else None
    _check(load_library().fp4_root_ns_static(G.data_ptr(), out.data_ptr(), m, n, steps, p,
                                             device_status.data_ptr() if device_status is not None else None,
                                             _stream(stream)), "fp4_root_ns_static")


def fp4_root_ns_batched_workspace_bytes(shapes, steps: int = 5, flags: int = 0) -> int:
    cnt = len(shapes)
    m = (C.c_int64 * cnt)(*[s[0] for s in shapes])
    n = (C.c_int64 * cnt)(*[s[1] for s in shapes])
    return int(load_library().fp4_root_ns_batched_workspace_bytes(cnt, m, n, steps, flags))


def fp4_root_ns_batched(Gs, outs, steps: int, params: NsParams | None, ws: torch.Tensor, stream=None) -> None:
    cnt = len(Gs)
    g = (C.c_void_p * cnt)(*[t.data_ptr() for t in Gs])
    o = (C.c_void_p * cnt)(*[t.data_ptr() for t in outs])
    m = (C.c_int64 * cnt)(*[t.shape[0] for t in Gs])
    n = (C.c_int64 * cnt)(*[t.shape[1] for t in Gs])
    p = C.byref(params) if params is not None else None
    _check(load_library().fp4_root_ns_batched(cnt, g, o, m, n, steps, p, ws.data_ptr(),
                                              ws.numel() * ws.element_size(), _stream(stream)),
           "fp4_root_ns_batched")


def fp4_last_device_status(ws: torch.Tensor, stream=None) -> int:
    return int(load_library().fp4_last_device_status(ws.data_ptr(), _stream(stream)))


def fp4_gemm_nt(a_codes, a_scales, a_sg: float, b_codes, b_scales, b_sg: float, D: torch.Tensor,
                status: torch.Tensor | None = None, stream=None) -> None:
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    _check(load_library().fp4_gemm_nt(a_codes.data_ptr(), a_scales.data_ptr(), float(a_sg), b_codes.data_ptr(),
                                      b_scales.data_ptr(), float(b_sg), M, N, K, D.data_ptr(),
                                      status.data_ptr() if status is not None else None, _stream(stream)),
           "fp4_gemm_nt")


def fp4_gemm_nt_resident(a_codes, a_scales, a_sg: float, b_codes, b_scales, b_sg: float, D: torch.Tensor,
                         status: torch.Tensor | None = None, stream=None) -> None:
    """The launch of fp4_gemm_nt with the operands fetched once per SM pair (tensor-pipe ceiling)."""
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    _check(load_library().fp4_gemm_nt_resident(a_codes.data_ptr(), a_scales.data_ptr(), float(a_sg),
                                               b_codes.data_ptr(), b_scales.data_ptr(), float(b_sg), M, N, K,
                                               D.data_ptr(), status.data_ptr() if status is not None else None,
                                               _stream(stream)),
           "fp4_gemm_nt_resident")


def fp4_profile_enable(on: bool) -> None:
    load_library().fp4_profile_enable(1 if on else 0)


def fp4_profile_collect():
    """{class name: (milliseconds, bracketed launch groups)} since the last collect."""
    n = len(PROF_CLASSES)
    ms = (C.c_float * n)()
    groups = (C.c_int * n)()
    _check(load_library().fp4_profile_collect(ms, groups), "fp4_profile_collect")
    return {PROF_CLASSES[i]: (float(ms[i]), int(groups[i])) for i in range(n)}


def fp4_selftest_bounded_wait(status: torch.Tensor, limit_us: int, stream=None) -> None:
    _check(load_library().fp4_selftest_bounded_wait(status.data_ptr(), int(limit_us), _stream(stream)),
           "fp4_selftest_bounded_wait")


def fp4_kernel_launches() -> int:
    return int(load_library().fp4_kernel_launches())
