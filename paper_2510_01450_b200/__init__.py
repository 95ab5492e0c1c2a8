"""B200-native Local Linear Attention: causal forward pass and single-query decode.

The compute lives in ``liblla.so`` (hand-written CUDA for sm_100a behind the C ABI of
``include/lla.h``).  ``binding`` marshals arguments to it; ``inputs`` holds the seeded synthetic
workloads; ``build`` compiles the library in-tree.
"""
from . import inputs  # noqa: F401
from .binding import (  # noqa: F401
    LLA_BF16, LLA_CG_PRECISE_ALL, LLA_CG_PRECISE_NONE, LLA_DEBUG_NO_LOADS, LLA_F32, LLA_IMPL_AUTO, LLA_IMPL_SIMT, LLA_IMPL_TENSOR, LLA_PHASE_ALL, LLA_PHASE_DIRECT,
    LLA_PHASE_ITERATIVE, LLA_STATUS_WORDS, STATUS_BAD_PIVOT, STATUS_ITER_SUM, STATUS_ROWS_AT_CAP, STATUS_TIMEOUT, LlaError,
    lla_decode, lla_decode_default_splits, lla_decode_ex, lla_decode_f32, lla_decode_host, lla_decode_noalloc,
    lla_decode_workspace_bytes, lla_forward, lla_forward_ex, lla_forward_f32, lla_forward_host,
    lla_forward_workspace_bytes, lla_version, status_string, lla_backward_ex, lla_backward_workspace_bytes,
)
