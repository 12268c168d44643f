"""NVFP4 Root Newton-Schulz step for B200 (sm_100a)."""
from . import workloads  # noqa: F401
