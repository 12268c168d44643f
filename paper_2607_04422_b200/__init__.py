"""NVFP4 Root Newton-Schulz step for B200 (sm_100a).

The product is the C-ABI library ``libfp4root.so`` built from ``csrc/``;
``binding`` is its thin ctypes front end and ``workloads`` the seeded synthetic
input generators.  There is no CPU fallback: every entry point raises if the
CUDA library is missing.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    FP4_FLAG_FOUR_SIX, FP4_FLAG_KEEP_OPERANDS, FP4_FLAG_NO_OUT, FP4_FLAG_OVERLAP_GROUPS, FP4_FLAG_RHT, FP4_FLAG_STORE_BF16, FP4_MOM_FLAG_SR, Fp4Error,
    AdamwParams, MomentumParams, NsParams, fp4_adamw_update, fp4_momentum_decode, fp4_momentum_update, fp4_gemm_nt, fp4_gemm_nt_resident, fp4_kernel_launches, fp4_profile_collect, fp4_profile_enable, fp4_last_device_status, fp4_quantize, fp4_root_coeffs, fp4_root_ns,
    fp4_root_ns_batched, fp4_root_ns_batched_workspace_bytes, fp4_root_ns_static, fp4_root_ns_workspace_bytes,
    fp4_root_ns_workspace_layout, fp4_scale_bytes, fp4_selftest_bounded_wait, fp4_status_string, library_path, load_library,
)
