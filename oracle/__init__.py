"""CPU oracle for the AcceptMoE verifier-side MoE layer.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg import this
package.  It is a thin ctypes/numpy wrapper around ``acm_oracle.cpp`` (plain C++,
no code shared with the CUDA library) and never touches a GPU.
"""
from .binding import (  # noqa: F401
    SelectParams,
    SelectStats,
    build,
    dequantize_mxfp4,
    expf,
    expert_ffn,
    logf,
    moe_verify,
    node_weights,
    route_restricted,
    router,
    select_eligible,
    tree_sum,
)
