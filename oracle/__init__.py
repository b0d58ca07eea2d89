"""CPU fp64 oracle for VORTA's routed attention.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library never does, and shares no code with it.
"""
from .vorta_oracle import (  # noqa: F401
    attn_coreset,
    attn_full,
    attn_sliding,
    build,
    coreset_len,
    coreset_select,
    num_threads,
    router_gates,
    soft_mixture,
    sta_block_mask,
    sta_token_mask,
)
