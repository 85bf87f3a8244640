"""Float64 CPU oracle for fused sigmoid self-attention.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this package:
only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
It shares no code with the CUDA implementation.
"""
from .sigattn_oracle import (  # noqa: F401
    sigmoid,
    causal_mask,
    position_bias,
    attention_weights,
    sigattn_fwd,
    sigattn_bwd,
    sigattn_bwd_dbias,
    sigattn_bwd_dtemp,
    sigattn_fwd_sequence_form,
    seqlen_norm,
)
