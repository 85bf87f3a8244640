"""ctypes binding of libsigattn.so: argument marshalling only.

Every step of the attention path runs inside the library's CUDA kernels.  PyTorch is
used for device memory and streams, nothing else.  There is no CPU or PyTorch
fallback: if the shared library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libsigattn.so")

DTYPE_BF16 = 0
DTYPE_FP32 = 1

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing. Build it with `python -m paper_2409_04431_b200.build` "
        "(needs nvcc); there is no fallback implementation."
    )

_lib = ctypes.CDLL(LIB_PATH)

_c = ctypes
_lib.sigattn_fwd.restype = _c.c_int
_lib.sigattn_fwd.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 4 + [_c.c_float, _c.c_float, _c.c_int,
                                                                    _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd.restype = _c.c_int
_lib.sigattn_bwd.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 4 + [_c.c_float, _c.c_float, _c.c_int,
                                                                    _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                    _c.c_size_t, _c.c_void_p]
_lib.sigattn_fwd_bias_vec.restype = _c.c_int
_lib.sigattn_fwd_bias_vec.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 4 + [_c.c_float, _c.c_void_p, _c.c_int,
                                                                             _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_bias_vec.restype = _c.c_int
_lib.sigattn_bwd_bias_vec.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 4 + [_c.c_float, _c.c_void_p, _c.c_int,
                                                                             _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                             _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_bwd_dtemp.restype = _c.c_int
_lib.sigattn_bwd_dtemp.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 4 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                          _c.c_void_p, _c.c_int, _c.c_void_p, _c.c_void_p,
                                                                          _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_bwd_shard_acc_kv.restype = _c.c_int
_lib.sigattn_bwd_shard_acc_kv.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p,
                                                                                 _c.c_int, _c.c_int, _c.c_void_p, _c.c_int,
                                                                                 _c.c_void_p, _c.c_void_p]
_lib.sigattn_check_cu_seqlens.restype = _c.c_int
_lib.sigattn_check_cu_seqlens.argtypes = [_c.c_void_p, _c.c_int, _c.c_int]
_lib.sigattn_peer_export.restype = _c.c_int
_lib.sigattn_peer_export.argtypes = [_c.c_void_p, _c.c_void_p, _c.POINTER(_c.c_size_t)]
_lib.sigattn_peer_open.restype = _c.c_int
_lib.sigattn_peer_open.argtypes = [_c.c_void_p, _c.c_size_t, _c.POINTER(_c.c_void_p)]
_lib.sigattn_peer_close.restype = _c.c_int
_lib.sigattn_peer_close.argtypes = [_c.c_void_p, _c.c_size_t]
_lib.sigattn_fwd_gqa.restype = _c.c_int
_lib.sigattn_fwd_gqa.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 5 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                        _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_gqa.restype = _c.c_int
_lib.sigattn_bwd_gqa.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 5 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                        _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                        _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_fwd_nk.restype = _c.c_int
_lib.sigattn_fwd_nk.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                       _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_nk.restype = _c.c_int
_lib.sigattn_bwd_nk.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                       _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                       _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_fwd_shard.restype = _c.c_int
_lib.sigattn_fwd_shard.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                          _c.c_int, _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_shard.restype = _c.c_int
_lib.sigattn_bwd_shard.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                          _c.c_int, _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                          _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_fwd_varlen.restype = _c.c_int
_lib.sigattn_fwd_varlen.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 5 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                           _c.c_void_p, _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_varlen.restype = _c.c_int
_lib.sigattn_bwd_varlen.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 5 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                           _c.c_void_p, _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                           _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_fwd_rowscale.restype = _c.c_int
_lib.sigattn_fwd_rowscale.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                             _c.c_void_p, _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_rowscale.restype = _c.c_int
_lib.sigattn_bwd_rowscale.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                             _c.c_void_p, _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                             _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_fwd_ragged.restype = _c.c_int
_lib.sigattn_fwd_ragged.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 4 + [_c.c_void_p, _c.c_int, _c.c_float, _c.c_float,
                                                                           _c.c_void_p, _c.c_int, _c.c_void_p, _c.c_int,
                                                                           _c.c_void_p]
_lib.sigattn_bwd_ragged.restype = _c.c_int
_lib.sigattn_bwd_ragged.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 4 + [_c.c_void_p, _c.c_int, _c.c_float, _c.c_float,
                                                                           _c.c_void_p, _c.c_int, _c.c_void_p, _c.c_int,
                                                                           _c.c_void_p, _c.c_void_p, _c.c_size_t, _c.c_void_p]
_lib.sigattn_fwd_shard_acc.restype = _c.c_int
_lib.sigattn_fwd_shard_acc.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p,
                                                                              _c.c_int, _c.c_int, _c.c_void_p, _c.c_int,
                                                                              _c.c_void_p]
_lib.sigattn_bwd_shard_acc.restype = _c.c_int
_lib.sigattn_bwd_shard_acc.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p,
                                                                              _c.c_int, _c.c_int, _c.c_void_p, _c.c_int,
                                                                              _c.c_void_p, _c.c_void_p]
_lib.sigattn_acc_to_bf16.restype = _c.c_int
_lib.sigattn_acc_to_bf16.argtypes = [_c.c_void_p, _c.c_void_p, _c.c_size_t, _c.c_float, _c.c_void_p]
_lib.sigattn_fwd_decode.restype = _c.c_int
_lib.sigattn_fwd_decode.argtypes = [_c.c_void_p] * 4 + [_c.c_int] * 6 + [_c.c_float, _c.c_float, _c.c_void_p, _c.c_int,
                                                                           _c.c_void_p, _c.c_int, _c.c_void_p, _c.c_size_t,
                                                                           _c.c_void_p]
_lib.sigattn_fwd_decode_workspace_bytes.restype = _c.c_size_t
_lib.sigattn_fwd_decode_workspace_bytes.argtypes = [_c.c_int] * 5
_lib.sigattn_seqlen_norm.restype = _c.c_int
_lib.sigattn_seqlen_norm.argtypes = [_c.c_void_p, _c.c_int, _c.c_int, _c.c_float, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_workspace_bytes.restype = _c.c_size_t
_lib.sigattn_bwd_workspace_bytes.argtypes = [_c.c_int] * 5
_lib.sigattn_step_host.restype = _c.c_int
_lib.sigattn_step_host.argtypes = [_c.c_void_p] * 8 + [_c.c_int] * 4 + [_c.c_float, _c.c_float, _c.c_int,
                                                                          _c.c_void_p, _c.c_int, _c.c_void_p,
                                                                          _c.c_size_t, _c.c_void_p]
_lib.sigattn_step_host_arena_bytes.restype = _c.c_size_t
_lib.sigattn_step_host_arena_bytes.argtypes = [_c.c_int] * 5
_lib.sigattn_bwd_set_timing_events.restype = _c.c_int
_lib.sigattn_bwd_set_timing_events.argtypes = [_c.c_void_p, _c.c_void_p]
_lib.sigattn_bwd_static_scratch.restype = _c.c_int
_lib.sigattn_bwd_static_scratch.argtypes = [_c.c_void_p] * 7 + [_c.c_int] * 4 + [_c.c_float, _c.c_float, _c.c_int,
                                                                                   _c.c_void_p, _c.c_int, _c.c_void_p]
_lib.sigattn_bwd_static_scratch_max_elements.restype = _c.c_size_t
_lib.sigattn_bwd_static_scratch_max_elements.argtypes = []
_lib.sigattn_selftest_bounded_wait.restype = _c.c_int
_lib.sigattn_selftest_bounded_wait.argtypes = [_c.c_int, _c.c_void_p]
_lib.sigattn_check.restype = _c.c_int
_lib.sigattn_check.argtypes = [_c.c_void_p]
_lib.sigattn_strerror.restype = _c.c_char_p
_lib.sigattn_strerror.argtypes = [_c.c_int]
_lib.sigattn_last_cuda_error.restype = _c.c_char_p
_lib.sigattn_last_cuda_error.argtypes = []
_lib.sigattn_version.restype = _c.c_int
_lib.sigattn_version.argtypes = []
_lib.sigattn_launch_count.restype = _c.c_ulonglong
_lib.sigattn_launch_count.argtypes = []

EXPORTED = [
    "sigattn_fwd", "sigattn_bwd", "sigattn_bwd_workspace_bytes", "sigattn_check",
    "sigattn_strerror", "sigattn_last_cuda_error", "sigattn_version", "sigattn_launch_count",
    "sigattn_step_host", "sigattn_step_host_arena_bytes", "sigattn_bwd_set_timing_events",
    "sigattn_bwd_static_scratch", "sigattn_bwd_static_scratch_max_elements",
    "sigattn_selftest_bounded_wait", "sigattn_fwd_bias_vec", "sigattn_bwd_bias_vec", "sigattn_bwd_dtemp",
    "sigattn_peer_export", "sigattn_peer_open", "sigattn_peer_close", "sigattn_bwd_shard_acc_kv", "sigattn_check_cu_seqlens",
    "sigattn_fwd_gqa", "sigattn_bwd_gqa", "sigattn_fwd_nk", "sigattn_bwd_nk",
    "sigattn_fwd_shard", "sigattn_bwd_shard", "sigattn_fwd_varlen", "sigattn_bwd_varlen",
    "sigattn_fwd_rowscale", "sigattn_bwd_rowscale", "sigattn_seqlen_norm",
    "sigattn_fwd_decode", "sigattn_fwd_decode_workspace_bytes",
    "sigattn_fwd_shard_acc", "sigattn_bwd_shard_acc", "sigattn_acc_to_bf16",
    "sigattn_fwd_ragged", "sigattn_bwd_ragged",
]


class SigattnError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        msg = _lib.sigattn_strerror(code).decode()
        if code == -7:
            msg += ": " + _lib.sigattn_last_cuda_error().decode()
        super().__init__(f"sigattn error {code}: {msg}")


def lib():
    """The loaded ctypes library (raw C-ABI access, e.g. for error-path tests)."""
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype == torch.float32:
        return DTYPE_FP32
    raise TypeError(f"sigattn supports bfloat16 and float32 tensors, got {t.dtype}")


def _slopes_ptr(alibi_slopes, q):
    """Device pointer of the per-head slopes after checking what the kernels rely on: float32, on q's
    device, contiguous, one slope per query head.  Anything else would make a kernel read a host
    address or past the end of the tensor, so it is refused here, before any launch."""
    if alibi_slopes is None:
        return None
    import torch
    H = q.shape[1]
    if (not isinstance(alibi_slopes, torch.Tensor) or not alibi_slopes.is_cuda or alibi_slopes.device != q.device
            or alibi_slopes.dtype != torch.float32 or not alibi_slopes.is_contiguous() or alibi_slopes.numel() != H):
        raise ValueError(f"alibi_slopes must be a contiguous float32 CUDA tensor of {H} slopes (one per query head) "
                         "on q's device")
    return alibi_slopes.data_ptr()


def _host_slopes_ptr(alibi_slopes, H):
    """Host pointer of the per-head slopes for sigattn_step_host, which copies them to the device itself."""
    if alibi_slopes is None:
        return None
    import torch
    if (not isinstance(alibi_slopes, torch.Tensor) or alibi_slopes.is_cuda or alibi_slopes.dtype != torch.float32
            or not alibi_slopes.is_contiguous() or alibi_slopes.numel() != H):
        raise ValueError(f"sigattn_step_host takes alibi_slopes as a contiguous float32 CPU tensor of {H} slopes")
    return alibi_slopes.data_ptr()


def _ws_ptr(workspace, q):
    """Device pointer of a caller-supplied scratch tensor: uint8, on q's device, contiguous."""
    if workspace is None:
        return None
    import torch
    if (not isinstance(workspace, torch.Tensor) or not workspace.is_cuda or workspace.device != q.device
            or workspace.dtype != torch.uint8 or not workspace.is_contiguous()):
        raise ValueError("workspace must be a contiguous uint8 CUDA tensor on q's device")
    return workspace.data_ptr()


def _check_same(ts, names):
    import torch
    ref = ts[0]
    if ref.dim() != 4:
        raise ValueError("tensors must be [B, H, N, D]")
    for t, n in zip(ts, names):
        if not isinstance(t, torch.Tensor) or not t.is_cuda:
            raise ValueError(f"{n} must be a CUDA tensor")
        if t.shape != ref.shape or t.dtype != ref.dtype or t.device != ref.device:
            raise ValueError(f"{n} must match q in shape, dtype and device")
        if not t.is_contiguous():
            raise ValueError(f"{n} must be contiguous [B, H, N, D]")


def sigattn_version() -> int:
    return _lib.sigattn_version()


def sigattn_launch_count() -> int:
    return int(_lib.sigattn_launch_count())


def sigattn_strerror(code: int) -> str:
    return _lib.sigattn_strerror(code).decode()


def sigattn_bwd_workspace_bytes(B, H, N, D, dtype_code) -> int:
    return int(_lib.sigattn_bwd_workspace_bytes(B, H, N, D, dtype_code))


def sigattn_check(stream=None) -> None:
    rc = _lib.sigattn_check(_stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)


def sigattn_fwd(q, k, v, scale, bias, causal=False, alibi_slopes=None, out=None, stream=None):
    """O = sigmoid(scale * Q K^T + bias [- slope * |i - j|]) [causal-masked] V.

    q, k, v: contiguous CUDA tensors [B, H, N, D], bfloat16 (tensor-core path) or
    float32 (debug path).  alibi_slopes: None or a float32 CUDA tensor of H slopes.
    Returns `out` (allocated if None).  Enqueues on the current stream; does not sync.
    """
    import torch
    _check_same([q, k, v], ["q", "k", "v"])
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    B, H, N, D = q.shape
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, D, float(scale), float(bias),
                              int(bool(causal)), _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None, workspace=None, out=None, stream=None):
    """(dQ, dK, dV) of L = sum(O * dO).  `workspace`: optional uint8 CUDA tensor of at
    least sigattn_bwd_workspace_bytes bytes (allocated if None).  `out`: optional
    (dq, dk, dv) tuple to write into."""
    import torch
    _check_same([q, k, v, d_o], ["q", "k", "v", "d_o"])
    B, H, N, D = q.shape
    code = _dtype_code(q)
    if out is None:
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    else:
        dq, dk, dv = out
        _check_same([q, dq, dk, dv], ["q", "dq", "dk", "dv"])
    need = sigattn_bwd_workspace_bytes(B, H, N, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, N, D,
                              float(scale), float(bias), int(bool(causal)), _slopes_ptr(alibi_slopes, q), code,
                              _ws_ptr(workspace, q), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv


def _check_bias_vec(bias_bh, q):
    import torch
    B, H = q.shape[0], q.shape[1]
    if (not isinstance(bias_bh, torch.Tensor) or not bias_bh.is_cuda or bias_bh.dtype != torch.float32
            or tuple(bias_bh.shape) != (B, H) or not bias_bh.is_contiguous() or bias_bh.device != q.device):
        raise ValueError("bias_bh must be a contiguous float32 CUDA tensor of shape [B, H] on q's device")


def sigattn_fwd_bias_vec(q, k, v, scale, bias_bh, causal=False, alibi_slopes=None, out=None, stream=None):
    """sigattn_fwd with one bias per (batch, head): `bias_bh` is a float32 CUDA tensor [B, H]."""
    import torch
    _check_same([q, k, v], ["q", "k", "v"])
    _check_bias_vec(bias_bh, q)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    B, H, N, D = q.shape
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_bias_vec(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, D, float(scale),
                                       _ptr(bias_bh), int(bool(causal)), _slopes_ptr(alibi_slopes, q), _dtype_code(q),
                                       _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd_bias_vec(q, k, v, d_o, scale, bias_bh, causal=False, alibi_slopes=None, want_dbias=True,
                         workspace=None, out=None, stream=None):
    """sigattn_bwd with the bias vector of sigattn_fwd_bias_vec.  Returns (dQ, dK, dV, dbias)
    where dbias is a float32 CUDA tensor [B, H] holding sum dS per (batch, head), or None if
    `want_dbias` is False."""
    import torch
    _check_same([q, k, v, d_o], ["q", "k", "v", "d_o"])
    _check_bias_vec(bias_bh, q)
    B, H, N, D = q.shape
    code = _dtype_code(q)
    if out is None:
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    else:
        dq, dk, dv = out
        _check_same([q, dq, dk, dv], ["q", "dq", "dk", "dv"])
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(B, H, N, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_bias_vec(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, N, D,
                                       float(scale), _ptr(bias_bh), int(bool(causal)), _slopes_ptr(alibi_slopes, q), code,
                                       _ptr(dbias), _ws_ptr(workspace, q), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dbias


def sigattn_bwd_dtemp(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None, want_dbias=False, workspace=None,
                      out=None, stream=None):
    """sigattn_bwd plus the gradient of a learnable temperature t in sigmoid(e^t * scale * Q K^T + b):
    pass scale * e^t as `scale`.  `bias`: a float, or a float32 CUDA tensor [B, H].  Returns
    (dQ, dK, dV, dtemp, dbias): dtemp is a float32 CUDA tensor [B, H] with sum_i <Q_i, dQ_i> per
    (batch, head) (sum it for a temperature shared by all heads); dbias as in sigattn_bwd_bias_vec, or
    None unless `want_dbias`."""
    import torch
    _check_same([q, k, v, d_o], ["q", "k", "v", "d_o"])
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    B, H, N, D = q.shape
    code = _dtype_code(q)
    if out is None:
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    else:
        dq, dk, dv = out
        _check_same([q, dq, dk, dv], ["q", "dq", "dk", "dv"])
    dtemp = torch.empty((B, H), dtype=torch.float32, device=q.device)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(B, H, N, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_dtemp(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, N, D,
                                    float(scale), 0.0 if vec else float(bias), _ptr(bias) if vec else None,
                                    int(bool(causal)), _slopes_ptr(alibi_slopes, q), code, _ptr(dbias), _ptr(dtemp),
                                    _ws_ptr(workspace, q), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dtemp, dbias


def _check_gqa(q, k, v):
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        if not isinstance(t, torch.Tensor) or not t.is_cuda or t.dim() != 4 or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous 4-D CUDA tensor")
    B, H, N, D = q.shape
    if k.shape != v.shape or k.shape[0] != B or k.shape[2] != N or k.shape[3] != D or k.dtype != q.dtype \
            or v.dtype != q.dtype or k.device != q.device or v.device != q.device:
        raise ValueError("k, v must be [B, H_kv, N, D] with q's B, N, D, dtype and device")
    return B, H, k.shape[1], N, D


def sigattn_fwd_gqa(q, k, v, scale, bias, causal=False, alibi_slopes=None, out=None, stream=None):
    """sigattn_fwd with k, v of H_kv <= H heads ([B, H_kv, N, D]); query head h reads head
    h // (H // H_kv).  `bias`: a float, or a float32 CUDA tensor [B, H]."""
    import torch
    B, H, H_kv, N, D = _check_gqa(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_gqa(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N, D, float(scale),
                                  0.0 if vec else float(bias), _ptr(bias) if vec else None, int(bool(causal)),
                                  _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd_gqa(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None, want_dbias=False, workspace=None,
                    stream=None):
    """Backward of sigattn_fwd_gqa.  Returns (dQ [B,H,N,D], dK, dV [B,H_kv,N,D], dbias or None)."""
    import torch
    B, H, H_kv, N, D = _check_gqa(q, k, v)
    _check_same([q, d_o], ["q", "d_o"])
    code = _dtype_code(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(B, H, N, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_gqa(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, H_kv, N, D,
                                  float(scale), 0.0 if vec else float(bias), _ptr(bias) if vec else None,
                                  int(bool(causal)), _slopes_ptr(alibi_slopes, q), code, _ptr(dbias), _ws_ptr(workspace, q), ws_bytes,
                                  _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dbias


def _check_nk(q, k, v):
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        if not isinstance(t, torch.Tensor) or not t.is_cuda or t.dim() != 4 or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous 4-D CUDA tensor")
    B, H, N_q, D = q.shape
    if k.shape != v.shape or k.shape[0] != B or k.shape[3] != D or k.dtype != q.dtype or v.dtype != q.dtype \
            or k.device != q.device or v.device != q.device:
        raise ValueError("k, v must be [B, H_kv, N_k, D] with q's B, D, dtype and device")
    return B, H, k.shape[1], N_q, k.shape[2], D


def sigattn_fwd_nk(q, k, v, scale, bias, causal=False, alibi_slopes=None, out=None, stream=None):
    """N_q queries against N_k keys: q [B, H, N_q, D], k, v [B, H_kv, N_k, D]; the queries are
    the last N_q positions (causal needs N_k >= N_q).  `bias`: float or float32 CUDA [B, H]."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_nk(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N_q, N_k, D, float(scale),
                                 0.0 if vec else float(bias), _ptr(bias) if vec else None, int(bool(causal)),
                                 _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd_nk(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None, want_dbias=False, workspace=None,
                   stream=None):
    """Backward of sigattn_fwd_nk.  Returns (dQ like q, dK like k, dV like v, dbias [B, H] or None)."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    _check_same([q, d_o], ["q", "d_o"])
    code = _dtype_code(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(B, H, N_q, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_nk(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, H_kv, N_q, N_k,
                                 D, float(scale), 0.0 if vec else float(bias), _ptr(bias) if vec else None,
                                 int(bool(causal)), _slopes_ptr(alibi_slopes, q), code, _ptr(dbias), _ws_ptr(workspace, q), ws_bytes,
                                 _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dbias


def sigattn_fwd_shard(q, k, v, scale, bias, pos0, causal=False, alibi_slopes=None, out=None, stream=None):
    """sigattn_fwd_nk against one contiguous shard of keys and values: `pos0` is the position
    of query row 0 minus the position of the shard's first key.  The results of all shards
    add up to the attention against the whole sequence."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_shard(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N_q, N_k, D, float(scale),
                                    0.0 if vec else float(bias), _ptr(bias) if vec else None, int(bool(causal)),
                                    int(pos0), _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd_shard(q, k, v, d_o, scale, bias, pos0, causal=False, alibi_slopes=None, want_dbias=False,
                      workspace=None, stream=None):
    """Backward of sigattn_fwd_shard: (dQ summand, dK, dV of the shard, dbias summand or None)."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    _check_same([q, d_o], ["q", "d_o"])
    code = _dtype_code(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(B, H, N_q, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_shard(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, H_kv, N_q,
                                    N_k, D, float(scale), 0.0 if vec else float(bias), _ptr(bias) if vec else None,
                                    int(bool(causal)), int(pos0), _slopes_ptr(alibi_slopes, q), code, _ptr(dbias),
                                    _ws_ptr(workspace, q), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dbias


def _check_seqlens(seqlens, q):
    import torch
    if (not isinstance(seqlens, torch.Tensor) or not seqlens.is_cuda or seqlens.dtype != torch.int32
            or tuple(seqlens.shape) != (q.shape[0],) or not seqlens.is_contiguous() or seqlens.device != q.device):
        raise ValueError("seqlens must be a contiguous int32 CUDA tensor of shape [B] on q's device")


def sigattn_fwd_varlen(q, k, v, scale, bias, seqlens, causal=False, alibi_slopes=None, out=None, stream=None):
    """Padded batch: `seqlens` (int32 CUDA [B]) gives the rows of each batch entry that count.
    `bias`: float or float32 CUDA [B, H] (e.g. -log of each length)."""
    import torch
    B, H, H_kv, N, D = _check_gqa(q, k, v)
    _check_seqlens(seqlens, q)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N, D, float(scale),
                                     0.0 if vec else float(bias), _ptr(bias) if vec else None, int(bool(causal)),
                                     _ptr(seqlens), _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd_varlen(q, k, v, d_o, scale, bias, seqlens, causal=False, alibi_slopes=None, want_dbias=False,
                       workspace=None, stream=None):
    """Backward of sigattn_fwd_varlen: (dQ, dK, dV, dbias or None); padded rows come out zero."""
    import torch
    B, H, H_kv, N, D = _check_gqa(q, k, v)
    _check_same([q, d_o], ["q", "d_o"])
    _check_seqlens(seqlens, q)
    code = _dtype_code(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(B, H, N, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, H_kv, N, D,
                                     float(scale), 0.0 if vec else float(bias), _ptr(bias) if vec else None,
                                     int(bool(causal)), _ptr(seqlens), _slopes_ptr(alibi_slopes, q), code, _ptr(dbias),
                                     _ws_ptr(workspace, q), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dbias


def _check_ragged(q, k, v, cu_seqlens, bias):
    import torch
    B, H, H_kv, T, D = _check_gqa(q, k, v)
    if B != 1:
        raise ValueError("a batch without padding has B = 1: q [1, H, T, D], k, v [1, H_kv, T, D]")
    if (not isinstance(cu_seqlens, torch.Tensor) or not cu_seqlens.is_cuda or cu_seqlens.dtype != torch.int32
            or cu_seqlens.dim() != 1 or cu_seqlens.numel() < 2 or not cu_seqlens.is_contiguous()
            or cu_seqlens.device != q.device):
        raise ValueError("cu_seqlens must be a contiguous int32 CUDA tensor of n_seqs + 1 row offsets on q's device")
    n_seqs = cu_seqlens.numel() - 1
    vec = isinstance(bias, torch.Tensor)
    if vec and (not bias.is_cuda or bias.dtype != torch.float32 or tuple(bias.shape) != (n_seqs, H)
                or not bias.is_contiguous() or bias.device != q.device):
        raise ValueError("bias must be a float or a contiguous float32 CUDA tensor [n_seqs, H] on q's device")
    return H, H_kv, T, D, n_seqs, vec


def sigattn_fwd_ragged(q, k, v, cu_seqlens, scale, bias, causal=False, alibi_slopes=None, out=None, stream=None):
    """Batch stored without padding: q [1, H, T, D], k, v [1, H_kv, T, D]; `cu_seqlens` int32 CUDA
    [n_seqs + 1] row offsets (rising from 0 to T; the caller's responsibility); `bias`: float or
    float32 CUDA [n_seqs, H]."""
    import torch
    H, H_kv, T, D, n_seqs, vec = _check_ragged(q, k, v, cu_seqlens, bias)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_ragged(_ptr(q), _ptr(k), _ptr(v), _ptr(out), H, H_kv, T, D, _ptr(cu_seqlens), n_seqs,
                                     float(scale), 0.0 if vec else float(bias), _ptr(bias) if vec else None,
                                     int(bool(causal)), _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd_ragged(q, k, v, d_o, cu_seqlens, scale, bias, causal=False, alibi_slopes=None, want_dbias=False,
                       workspace=None, stream=None):
    """Backward of sigattn_fwd_ragged: (dQ, dK, dV, dbias [n_seqs, H] or None)."""
    import torch
    H, H_kv, T, D, n_seqs, vec = _check_ragged(q, k, v, cu_seqlens, bias)
    _check_same([q, d_o], ["q", "d_o"])
    code = _dtype_code(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    dbias = torch.empty((n_seqs, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(1, H, T, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_ragged(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), H, H_kv, T, D,
                                     _ptr(cu_seqlens), n_seqs, float(scale), 0.0 if vec else float(bias),
                                     _ptr(bias) if vec else None, int(bool(causal)), _slopes_ptr(alibi_slopes, q), code,
                                     _ptr(dbias), _ws_ptr(workspace, q), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dbias


def sigattn_fwd_shard_acc(q, k, v, o_acc, scale, bias, pos0, causal=False, alibi_slopes=None, stream=None):
    """Adds this key/value shard's summand of O, in fp32, into `o_acc`: a float32 CUDA tensor shaped
    like q, or an integer device address (e.g. a peer mapping of another GPU's accumulator)."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    if isinstance(o_acc, torch.Tensor) and (o_acc.dtype != torch.float32 or o_acc.shape != q.shape
                                            or not o_acc.is_contiguous() or not o_acc.is_cuda):
        raise ValueError("o_acc must be a contiguous float32 CUDA tensor shaped like q")
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_shard_acc(_ptr(q), _ptr(k), _ptr(v), _ptr(o_acc), B, H, H_kv, N_q, N_k, D, float(scale),
                                        0.0 if vec else float(bias), _ptr(bias) if vec else None, int(bool(causal)),
                                        int(pos0), _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)


def sigattn_bwd_shard_acc(q, k, v, d_o, dq_acc, scale, bias, pos0, causal=False, alibi_slopes=None, want_dbias=False,
                          stream=None):
    """Adds this shard's summand of dQ (without the factor `scale`) into `dq_acc` (float32 CUDA tensor
    shaped like q, or an integer device address) and returns (dK, dV, dbias or None) of the shard."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    _check_same([q, d_o], ["q", "d_o"])
    if isinstance(dq_acc, torch.Tensor) and (dq_acc.dtype != torch.float32 or dq_acc.shape != q.shape
                                             or not dq_acc.is_contiguous() or not dq_acc.is_cuda):
        raise ValueError("dq_acc must be a contiguous float32 CUDA tensor shaped like q")
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    dk, dv = torch.empty_like(k), torch.empty_like(v)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_shard_acc(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq_acc), _ptr(dk), _ptr(dv), B, H,
                                        H_kv, N_q, N_k, D, float(scale), 0.0 if vec else float(bias),
                                        _ptr(bias) if vec else None, int(bool(causal)), int(pos0), _slopes_ptr(alibi_slopes, q),
                                        _dtype_code(q), _ptr(dbias), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dk, dv, dbias


def sigattn_bwd_shard_acc_kv(q, k, v, d_o, dq_acc, dk, dv, scale, bias, pos0, causal=False, alibi_slopes=None,
                             want_dbias=False, stream=None):
    """sigattn_bwd_shard_acc that ADDS the shard's dK, dV into the given bf16 tensors `dk`, `dv` (shaped
    like k, v; cleared by the caller before the first call) instead of returning new ones: the sum over
    several calls (one per owner of query rows) forms inside the library.  Returns dbias or None."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    _check_same([q, d_o], ["q", "d_o"])
    _check_same([k, dk, dv], ["k", "dk", "dv"])
    if isinstance(dq_acc, torch.Tensor) and (dq_acc.dtype != torch.float32 or dq_acc.shape != q.shape
                                             or not dq_acc.is_contiguous() or not dq_acc.is_cuda):
        raise ValueError("dq_acc must be a contiguous float32 CUDA tensor shaped like q")
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_shard_acc_kv(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq_acc), _ptr(dk), _ptr(dv), B,
                                           H, H_kv, N_q, N_k, D, float(scale), 0.0 if vec else float(bias),
                                           _ptr(bias) if vec else None, int(bool(causal)), int(pos0),
                                           _slopes_ptr(alibi_slopes, q), _dtype_code(q), _ptr(dbias), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dbias


def sigattn_acc_to_bf16(acc, mul=1.0, out=None, stream=None):
    """bf16(mul * acc) for a float32 accumulator filled by the *_shard_acc calls."""
    import torch
    if not isinstance(acc, torch.Tensor) or acc.dtype != torch.float32 or not acc.is_cuda or not acc.is_contiguous():
        raise ValueError("acc must be a contiguous float32 CUDA tensor")
    if out is None:
        out = torch.empty(acc.shape, dtype=torch.bfloat16, device=acc.device)
    with torch.cuda.device(acc.device):
        rc = _lib.sigattn_acc_to_bf16(_ptr(acc), _ptr(out), acc.numel(), float(mul), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_fwd_decode_workspace_bytes(B, H, N_q, D, dtype_code) -> int:
    return int(_lib.sigattn_fwd_decode_workspace_bytes(B, H, N_q, D, dtype_code))


def sigattn_fwd_decode(q, k, v, scale, bias, causal=False, alibi_slopes=None, workspace=None, out=None, stream=None):
    """sigattn_fwd_nk with a scratch buffer that lets the keys of one head be split over several
    thread blocks (generation with a cache: few queries, long key sequences)."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    code = _dtype_code(q)
    need = sigattn_fwd_decode_workspace_bytes(B, H, N_q, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_decode(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N_q, N_k, D, float(scale),
                                     0.0 if vec else float(bias), _ptr(bias) if vec else None, int(bool(causal)),
                                     _slopes_ptr(alibi_slopes, q), code, _ws_ptr(workspace, q), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def _check_row_scale(row_scale, q):
    import torch
    if (not isinstance(row_scale, torch.Tensor) or not row_scale.is_cuda or row_scale.dtype != torch.float32
            or tuple(row_scale.shape) != (q.shape[2],) or not row_scale.is_contiguous()
            or row_scale.device != q.device):
        raise ValueError("row_scale must be a contiguous float32 CUDA tensor of shape [N_q] on q's device")


def sigattn_seqlen_norm(n_q, n_k, alpha, causal, device, stream=None):
    """The paper's row factors of the sequence-length normalisation as a float32 CUDA [n_q]:
    n_k^-alpha without a mask, (position + 1)^-alpha with the causal mask."""
    import torch
    out = torch.empty(int(n_q), dtype=torch.float32, device=device)
    with torch.cuda.device(out.device):
        rc = _lib.sigattn_seqlen_norm(_ptr(out), int(n_q), int(n_k), float(alpha), int(bool(causal)),
                                      _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_fwd_rowscale(q, k, v, scale, bias, row_scale, causal=False, alibi_slopes=None, out=None, stream=None):
    """O_i = row_scale[i] * sum_j P_ij V_j (sequence-length normalisation); q [B, H, N_q, D], k, v
    [B, H_kv, N_k, D]; `bias`: float or float32 CUDA [B, H]."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    _check_row_scale(row_scale, q)
    if out is None:
        out = torch.empty_like(q)
    else:
        _check_same([q, out], ["q", "out"])
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_fwd_rowscale(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, H_kv, N_q, N_k, D, float(scale),
                                       0.0 if vec else float(bias), _ptr(bias) if vec else None, int(bool(causal)),
                                       _ptr(row_scale), _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return out


def sigattn_bwd_rowscale(q, k, v, d_o, scale, bias, row_scale, causal=False, alibi_slopes=None, want_dbias=False,
                         workspace=None, stream=None):
    """Backward of sigattn_fwd_rowscale: (dQ, dK, dV, dbias or None)."""
    import torch
    B, H, H_kv, N_q, N_k, D = _check_nk(q, k, v)
    _check_same([q, d_o], ["q", "d_o"])
    _check_row_scale(row_scale, q)
    code = _dtype_code(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    vec = isinstance(bias, torch.Tensor)
    if vec:
        _check_bias_vec(bias, q)
    dbias = torch.empty((B, H), dtype=torch.float32, device=q.device) if want_dbias else None
    need = sigattn_bwd_workspace_bytes(B, H, N_q, D, code)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_rowscale(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, H_kv,
                                       N_q, N_k, D, float(scale), 0.0 if vec else float(bias),
                                       _ptr(bias) if vec else None, int(bool(causal)), _ptr(row_scale),
                                       _slopes_ptr(alibi_slopes, q), code, _ptr(dbias), _ws_ptr(workspace, q), ws_bytes,
                                       _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv, dbias


def sigattn_step_host_arena_bytes(B, H, N, D, dtype_code) -> int:
    return int(_lib.sigattn_step_host_arena_bytes(B, H, N, D, dtype_code))


def sigattn_step_host(q, k, v, d_o, o, dq, dk, dv, scale, bias, causal=False, alibi_slopes=None, arena=None,
                      stream=None):
    """Forward + backward from HOST tensors (CPU torch tensors, ideally pinned): copies the
    inputs to the device, runs both passes, copies O, dQ, dK, dV back into the given host
    tensors; everything is enqueued on the current stream and nothing is synchronised.
    `arena`: uint8 CUDA tensor of at least sigattn_step_host_arena_bytes bytes.
    `alibi_slopes`: None or a float32 CPU tensor of H slopes."""
    import torch
    ts = [q, k, v, d_o, o, dq, dk, dv]
    for t in ts:
        if t.is_cuda or not t.is_contiguous() or t.shape != q.shape or t.dtype != q.dtype:
            raise ValueError("sigattn_step_host takes contiguous CPU tensors of one shape and dtype")
    B, H, N, D = q.shape
    code = _dtype_code(q)
    need = sigattn_step_host_arena_bytes(B, H, N, D, code)
    if arena is None:
        arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    with torch.cuda.device(arena.device):
        rc = _lib.sigattn_step_host(*[_ptr(t) for t in ts], B, H, N, D, float(scale), float(bias),
                                    int(bool(causal)), _host_slopes_ptr(alibi_slopes, H), code, _ptr(arena),
                                    arena.numel(), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return arena


def sigattn_bwd_set_timing_events(start=None, stop=None) -> None:
    """start, stop: torch.cuda.Event(enable_timing=True) that have been recorded once
    (so that their handles exist), or None, None to switch the hook off."""
    a = None if start is None else start.cuda_event
    b = None if stop is None else stop.cuda_event
    _lib.sigattn_bwd_set_timing_events(a, b)


def sigattn_bwd_static_scratch_max_elements() -> int:
    return int(_lib.sigattn_bwd_static_scratch_max_elements())


def sigattn_bwd_static_scratch(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None, out=None, stream=None):
    """sigattn_bwd for callers that must not allocate device memory: the fp32 dQ
    accumulator is a fixed array inside the library, so no workspace is passed (and this
    wrapper allocates none; give `out=(dq, dk, dv)` to avoid even the output allocation).
    B*H*N*D is limited to sigattn_bwd_static_scratch_max_elements(); calls that overlap on
    the device share the array and race, so keep them on one stream."""
    import torch
    _check_same([q, k, v, d_o], ["q", "k", "v", "d_o"])
    B, H, N, D = q.shape
    if out is None:
        dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    else:
        dq, dk, dv = out
        _check_same([q, dq, dk, dv], ["q", "dq", "dk", "dv"])
    with torch.cuda.device(q.device):
        rc = _lib.sigattn_bwd_static_scratch(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv),
                                             B, H, N, D, float(scale), float(bias), int(bool(causal)),
                                             _slopes_ptr(alibi_slopes, q), _dtype_code(q), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
    return dq, dk, dv


def sigattn_check_cu_seqlens(cu_seqlens_host, T: int) -> None:
    """Raise SigattnError(-2) unless the HOST int32 tensor `cu_seqlens_host` (n_seqs + 1 offsets) starts at 0,
    never decreases and ends at T.  The ragged kernels trust the device copy; this is the check a caller
    can run on its host copy before launching."""
    import torch
    if (not isinstance(cu_seqlens_host, torch.Tensor) or cu_seqlens_host.is_cuda or cu_seqlens_host.dtype != torch.int32
            or not cu_seqlens_host.is_contiguous() or cu_seqlens_host.numel() < 2):
        raise ValueError("cu_seqlens_host must be a contiguous int32 CPU tensor of n_seqs + 1 offsets")
    rc = _lib.sigattn_check_cu_seqlens(cu_seqlens_host.data_ptr(), cu_seqlens_host.numel() - 1, int(T))
    if rc != 0:
        raise SigattnError(rc)


PEER_HANDLE_BYTES = 64


def sigattn_peer_export(t):
    """Handle for the allocation that holds CUDA tensor `t` plus the offset of t's first byte in it:
    (bytes, int), to be sent to the other processes over any host channel (see sigattn_peer_open)."""
    buf = _c.create_string_buffer(PEER_HANDLE_BYTES)
    off = _c.c_size_t(0)
    with __import__("torch").cuda.device(t.device):
        rc = _lib.sigattn_peer_export(_ptr(t), buf, _c.byref(off))
    if rc != 0:
        raise SigattnError(rc)
    return bytes(buf.raw), int(off.value)


def sigattn_peer_open(handle: bytes, offset: int, device=None) -> int:
    """Map another process's exported allocation on `device` (default: the current one) and return
    the device address that corresponds to the exported tensor's first byte.  Pass it where the shard
    calls take an accumulator; close it with sigattn_peer_close(address, offset)."""
    import torch
    out = _c.c_void_p(0)
    with torch.cuda.device(torch.cuda.current_device() if device is None else device):
        rc = _lib.sigattn_peer_open(handle, int(offset), _c.byref(out))
    if rc != 0:
        raise SigattnError(rc)
    return int(out.value)


def sigattn_peer_close(address: int, offset: int) -> None:
    rc = _lib.sigattn_peer_close(_c.c_void_p(address), int(offset))
    if rc != 0:
        raise SigattnError(rc)


def sigattn_selftest_bounded_wait(limit_us: int = 2000, stream=None) -> None:
    """Enqueue the failure-path self-test: a kernel whose bounded wait must expire after
    `limit_us` microseconds.  The following sigattn_check() raises SigattnError(-8)."""
    rc = _lib.sigattn_selftest_bounded_wait(int(limit_us), _stream_ptr(stream))
    if rc != 0:
        raise SigattnError(rc)
