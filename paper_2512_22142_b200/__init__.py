"""Cleave hot path on one B200: plan -> grouped sub-GEMM execution -> assembly -> reissue.

Thin ctypes binding over the C-ABI library `lib/libcleave.so` (CUDA kernels for sm_100a).  The
binding only marshals arguments; every step runs in the library.  There is no fallback: if the
library has not been built, importing this package raises.
"""
from .binding import (CleaveError, Plan, default_opts, lib, lib_path, plan, plan_uniform,  # noqa: F401
                      GEMM_DTYPE, TASK_DTYPE, DEVICE_DTYPE, strerror)
