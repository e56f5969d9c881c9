"""B200-native COMP-AMS optimizer step (Algorithm 2 of "On Distributed Adaptive Optimization
with Gradient Compression"): hand-written sm_100a CUDA kernels behind a C ABI, plus a thin
ctypes binding. The CUDA library is loaded on first use and its absence is an error: there is
no CPU fallback."""

from .binding import (  # noqa: F401
    BLOCKSIGN,
    RANDK,
    TOPK,
    CompAMS,
    CompAMSError,
    library_path,
    load_library,
    workspace_bytes,
)
