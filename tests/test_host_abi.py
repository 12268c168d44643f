"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its
host logic (coefficients, workspace sizes, argument validation) behaves; no kernels run."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "fp4root.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fp4_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2607_04422_b200 import build
    build.build()
    lib = ctypes.CDLL(fp4.library_path())
    names = _declared_symbols()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings():
    assert fp4.fp4_status_string(0) == "ok"
    for code in range(1, 9):
        assert fp4.fp4_status_string(code) not in ("", "unknown status")


def test_coefficients_match_the_oracle_provider():
    for m, n in ((256, 512), (3072, 3072), (3072, 8192), (8192, 3072), (2048, 8192)):
        assert fp4.fp4_root_coeffs(m, n) == oracle.root_coeffs(m, n)


def test_scale_bytes_and_workspace_sizes():
    assert fp4.fp4_scale_bytes(128, 128) == 1024
    assert fp4.fp4_scale_bytes(256, 512) == 2 * 8 * 512
    assert fp4.fp4_root_ns_workspace_bytes(100, 128) == 0
    # multiples of 16 are padded to multiples of 128 inside the workspace
    assert fp4.fp4_root_ns_workspace_bytes(144, 272, 5) == fp4.fp4_root_ns_workspace_bytes(256, 384, 5)
    assert fp4.fp4_root_ns_workspace_bytes(16, 16, 5) == fp4.fp4_root_ns_workspace_bytes(128, 128, 5)
    assert fp4.fp4_root_ns_workspace_bytes(136, 128, 5) == 0                      # not a multiple of 16
    small = fp4.fp4_root_ns_workspace_bytes(128, 256, 5)
    big = fp4.fp4_root_ns_workspace_bytes(3072, 8192, 5)
    assert 0 < small < big
    assert fp4.fp4_root_ns_workspace_bytes(8192, 3072, 5) == big + 3072 * 8192 * 4  # tall: X lives in the workspace
    both = fp4.fp4_root_ns_batched_workspace_bytes([(128, 256), (3072, 8192)], 5)
    assert both >= small + big and both < small + big + (1 << 16)  # one workspace per matrix
    # flag bits the library does not know are an error, not ignored: the size query answers 0
    assert fp4.fp4_root_ns_workspace_bytes(128, 256, 5, 64) == 0
    assert fp4.fp4_root_ns_workspace_bytes(128, 256, 5, fp4.FP4_FLAG_OVERLAP_GROUPS) == small  # the newest known bit
    assert fp4.fp4_root_ns_workspace_bytes(128, 256, 5, 0xABCD0000) == 0
    assert fp4.fp4_root_ns_batched_workspace_bytes([(128, 256)], 5, 1 << 20) == 0
    lay = fp4.fp4_root_ns_workspace_layout(512, 256, 5)
    offs = [lay.header, lay.scalars, lay.X, lay.A, lay.qX_codes, lay.qX_scales, lay.qXt_codes[0],
            lay.qXt_scales[0], lay.qXt_codes[1], lay.qXt_scales[1], lay.qA_codes, lay.qA_scales,
            lay.qB_codes, lay.qB_scales, lay.total]
    assert offs == sorted(offs) and all(o % 1024 == 0 for o in offs)


def test_argument_validation_happens_before_any_device_work():
    lib = fp4.load_library()
    buf = (ctypes.c_uint8 * 4096)()
    p = ctypes.addressof(buf)
    p = (p + 1023) // 1024 * 1024  # an aligned host address: never dereferenced by these calls
    assert lib.fp4_root_ns(None, p, 128, 128, 5, None, p, 1 << 30, None) == 1     # null input
    assert lib.fp4_root_ns(p, p, 100, 128, 5, None, p, 1 << 30, None) == 2        # shape
    assert lib.fp4_root_ns(p, p, 128, 128, 65, None, p, 1 << 30, None) == 1       # steps
    assert lib.fp4_root_ns(p + 4, p, 128, 128, 5, None, p, 1 << 30, None) == 3    # alignment
    assert lib.fp4_root_ns(p, p, 128, 128, 5, None, p + 128, 1 << 30, None) == 3  # workspace alignment
    assert lib.fp4_root_ns(p, p, 128, 128, 5, None, p, 16, None) == 4             # workspace
    assert lib.fp4_quantize(p, 128, 120, p, p, p, 0, None) == 2
    assert lib.fp4_gemm_nt(p, p, 1.0, p, p, 1.0, 128, 128, 64, p, None, None) == 2
    # the optimiser-state entry points
    mp = binding.MomentumParams(0.9, 1.0, 0, 0, 0)
    assert lib.fp4_momentum_update(None, 16, 16, p, p, None, None, ctypes.byref(mp), None) == 1   # null input
    assert lib.fp4_momentum_update(p, 16, 24, p, p, None, None, ctypes.byref(mp), None) == 2      # shape
    assert lib.fp4_momentum_update(p + 16, 16, 16, p, p, None, None, ctypes.byref(mp), None) == 3  # 32-byte rule
    bad = binding.MomentumParams(0.9, 1.0, 8, 0, 0)
    assert lib.fp4_momentum_update(p, 16, 16, p, p, None, None, ctypes.byref(bad), None) == 1     # unknown flag
    assert lib.fp4_momentum_decode(p, p, 16, 16, None, None) == 1
    ap = binding.AdamwParams(1e-3, 0.9, 0.95, 1e-8, 0.1, 1, 0, 0, 0)
    assert lib.fp4_adamw_update(p, p, 384, p, p, p, p, p, ctypes.byref(ap), None) == 2            # not a multiple of 256
    assert lib.fp4_adamw_update(p + 16, p, 256, p, p, p, p, p, ctypes.byref(ap), None) == 3
    ap0 = binding.AdamwParams(1e-3, 0.9, 0.95, 1e-8, 0.1, 0, 0, 0, 0)
    assert lib.fp4_adamw_update(p, p, 256, p, p, p, p, p, ctypes.byref(ap0), None) == 1           # step < 1


def test_no_gpu_on_the_optimiser_state_entry_points():
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for machines without a GPU")
    lib = fp4.load_library()
    buf = (ctypes.c_uint8 * (1 << 16))()
    p = (ctypes.addressof(buf) + 1023) // 1024 * 1024
    mp = binding.MomentumParams(0.9, 1.0, 0, 0, 0)
    assert lib.fp4_momentum_update(p, 16, 16, p, p, None, None, ctypes.byref(mp), None) in (5, 6)
    ap = binding.AdamwParams(1e-3, 0.9, 0.95, 1e-8, 0.1, 1, 0, 0, 0)
    assert lib.fp4_adamw_update(p, p, 256, p, p, p, p, p, ctypes.byref(ap), None) in (5, 6)


def test_no_gpu_means_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for machines without a GPU")
    lib = fp4.load_library()
    buf = (ctypes.c_uint8 * (1 << 20))()
    p = (ctypes.addressof(buf) + 1023) // 1024 * 1024
    rc = lib.fp4_quantize(p, 128, 128, p, p, p, 0, None)
    assert rc in (5, 6)  # FP4_ERR_ARCH or FP4_ERR_CUDA: nothing is computed on the CPU


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()
    monkeypatch.undo()
    binding.load_library()
