"""Fused sigmoid self-attention (forward + backward) for NVIDIA B200.

The computation lives in libsigattn.so (hand-written CUDA for sm_100a, C ABI declared
in include/sigattn.h).  This package is the thin Python binding plus the seeded
synthetic-input recipes used by the tests and the benchmark.

The binding is imported on first use of one of its names, so that
`python -m paper_2409_04431_b200.build` can run before the library exists; using any
operation without the built library raises ImportError (there is no fallback).
"""
_BINDING_NAMES = (
    "DTYPE_BF16",
    "DTYPE_FP32",
    "SigattnError",
    "sigattn_bwd",
    "sigattn_bwd_workspace_bytes",
    "sigattn_check",
    "sigattn_fwd",
    "sigattn_launch_count",
    "sigattn_strerror",
    "sigattn_version",
    "sigattn_step_host",
    "sigattn_step_host_arena_bytes",
    "sigattn_bwd_set_timing_events",
    "sigattn_bwd_static_scratch",
    "sigattn_bwd_static_scratch_max_elements",
    "sigattn_selftest_bounded_wait",
    "sigattn_fwd_bias_vec",
    "sigattn_bwd_bias_vec",
    "sigattn_bwd_dtemp",
    "sigattn_fwd_gqa",
    "sigattn_bwd_gqa",
    "sigattn_fwd_nk",
    "sigattn_bwd_nk",
    "sigattn_fwd_shard",
    "sigattn_bwd_shard",
    "sigattn_fwd_varlen",
    "sigattn_bwd_varlen",
    "sigattn_fwd_rowscale",
    "sigattn_bwd_rowscale",
    "sigattn_seqlen_norm",
    "sigattn_fwd_decode",
    "sigattn_fwd_shard_acc",
    "sigattn_bwd_shard_acc",
    "sigattn_bwd_shard_acc_kv",
    "sigattn_acc_to_bf16",
    "sigattn_peer_export",
    "sigattn_peer_open",
    "sigattn_peer_close",
    "sigattn_fwd_ragged",
    "sigattn_bwd_ragged",
    "sigattn_check_cu_seqlens",
    "sigattn_fwd_decode_workspace_bytes",
    "lib",
)

__all__ = list(_BINDING_NAMES)


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
