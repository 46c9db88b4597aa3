"""B200-native BitDelta fused GEMM: Y_b = X_b W_base^T + alpha_b (X_b S_b^T).

The work is done by hand-written sm_100a CUDA kernels behind a C-ABI shared
library (``libbitdelta.so``, declared in ``include/bitdelta.h``).  This package
is the thin Python binding (argument marshalling only) plus the seeded input
generators.  There is no CPU fallback: every call raises if the library is
missing.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    STATUS_RANGE,
    STATUS_TIMEOUT,
    BitDeltaError,
    compress,
    gemm,
    gemm_host,
    gemm_host_arena_bytes,
    gemm_noalloc,
    gemm_plan,
    gemm_plan_cta_items,
    gemm_plan_item_cta,
    gemm_workspace_bytes,
    kernel_launch_count,
    last_device_status,
    library_path,
    load_library,
    make_workspace,
    pack,
    selftest_timeout,
    status_string,
    unpack,
)
