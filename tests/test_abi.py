"""Host-only checks of the C-ABI library: it loads without a GPU, exports every symbol
the header declares, validates arguments before touching a device, and the Python
binding marshals to the same names."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "sigattn.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2409_04431_b200 import build
    build.build()
    from paper_2409_04431_b200 import binding
    return binding.lib()


def declared_symbols():
    text = open(HEADER).read()
    return re.findall(r"SIGATTN_API\s+[\w\s\*]+?\b(sigattn_\w+)\s*\(", text)


def test_header_declares_the_boundary():
    names = declared_symbols()
    for required in ("sigattn_fwd", "sigattn_bwd", "sigattn_bwd_workspace_bytes", "sigattn_check",
                     "sigattn_strerror", "sigattn_version"):
        assert required in names


def test_library_exports_every_declared_symbol(lib):
    from paper_2409_04431_b200 import binding
    for name in declared_symbols():
        assert hasattr(lib, name), name
        assert name in binding.EXPORTED, name
    raw = ctypes.CDLL(binding.LIB_PATH)
    for name in declared_symbols():
        getattr(raw, name)


def test_version_and_error_strings(lib):
    assert lib.sigattn_version() >= 100
    seen = set()
    for code in range(0, -9, -1):
        s = lib.sigattn_strerror(code).decode()
        assert s and s not in seen
        seen.add(s)
    assert "unknown" in lib.sigattn_strerror(-99).decode()


def test_workspace_bytes(lib):
    # fp32 dQ accumulator [B, H, N, D] at least; 0 for the fp32 path and for bad shapes
    assert lib.sigattn_bwd_workspace_bytes(2, 16, 4096, 128, 0) >= 2 * 16 * 4096 * 128 * 4
    assert lib.sigattn_bwd_workspace_bytes(2, 16, 4096, 128, 1) == 0
    assert lib.sigattn_bwd_workspace_bytes(2, 16, 4096, 96, 0) == 0
    assert lib.sigattn_bwd_workspace_bytes(0, 16, 4096, 128, 0) == 0


def test_argument_validation_happens_before_any_device_work(lib):
    """These calls must return their error codes on a machine without a GPU."""
    buf = np.zeros(4096, dtype=np.uint8)
    p = buf.ctypes.data
    p = (p + 255) & ~255
    ok = dict(B=1, H=1, N=4, D=64)
    f = lib.sigattn_fwd
    assert f(None, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, None) == -1
    assert f(p, p, p, None, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, None) == -1
    assert f(p, p, p, p, 1, 1, 4, 96, 0.125, 0.0, 0, None, 0, None) == -2
    assert f(p, p, p, p, 1, 1, 0, 64, 0.125, 0.0, 0, None, 0, None) == -2
    assert f(p, p, p, p, 0, 1, 4, 64, 0.125, 0.0, 0, None, 0, None) == -2
    assert f(p, p, p, p, 70000, 1, 4, 64, 0.125, 0.0, 0, None, 0, None) == -2
    assert f(p + 2, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, None) == -3
    assert f(p, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 0, None, 7, None) == -4
    assert f(p, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 2, None, 0, None) == -4
    g = lib.sigattn_bwd
    assert g(p, p, p, p, p, p, None, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, p, 4096, None) == -1
    assert g(p, p, p, p, p, p, p, 1, 1, 4, 48, 0.125, 0.0, 0, None, 0, p, 4096, None) == -2
    assert g(p, p, p, p, p, p, p + 8, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, p, 4096, None) == -3
    assert g(p, p, p, p, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, None, 0, None) == -1      # workspace missing
    assert g(p, p, p, p, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, p + 16, 4096, None) == -3  # workspace alignment
    assert g(p, p, p, p, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 0, None, 0, p, 16, None) == -5
    assert g(p, p, p, p, p, p, p, 1, 1, 4, 64, 0.125, 0.0, 0, None, 3, p, 4096, None) == -4


def test_input_recipes():
    from paper_2409_04431_b200 import inputs
    cfg = inputs.CONFIGS["c4"]
    q, k, v, d_o = inputs.make_inputs(cfg, heads=1, batch=1)
    assert q.shape == (1, 1, 4096, 128) and q.dtype == np.float32
    # qk-norm recipe: rows of q, k have L2 norm sqrt(D) up to bf16 rounding
    np.testing.assert_allclose(np.linalg.norm(q, axis=-1), math.sqrt(128), rtol=2e-3)
    np.testing.assert_allclose(np.linalg.norm(k, axis=-1), math.sqrt(128), rtol=2e-3)
    # values are exactly representable in bf16, and the generator is reproducible
    for t in (q, k, v, d_o):
        np.testing.assert_array_equal(inputs.round_to_bf16(t), t)
    q2, *_ = inputs.make_inputs(cfg, heads=1, batch=1)
    np.testing.assert_array_equal(q, q2)
    c3 = inputs.CONFIGS["c3"]
    np.testing.assert_allclose(c3.slopes(), [2.0 ** (-8 * h / 16) for h in range(1, 17)], rtol=1e-6)
    assert abs(inputs.CONFIGS["c5"].bias + math.log(16384)) < 1e-12
    # FLOP model: c = (n + 1) / (2 n) equals the unmasked fraction of the n x n matrix
    n = 37
    assert inputs.causal_fraction(n, True) == np.tril(np.ones((n, n))).sum() / n ** 2
    assert cfg.flops_fwd() == 4 * inputs.causal_fraction(4096, True) * 2 * 16 * 4096 ** 2 * 128
    assert cfg.flops_bwd() == 2.5 * cfg.flops_fwd()


def test_bf16_rounding_is_round_to_nearest_even():
    from paper_2409_04431_b200 import inputs
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.14159, 1e-30, 65504.0], dtype=np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    back = inputs.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert back[1] == 1.0 and back[2] == 1.015625
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    try:
        import torch
        t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
        np.testing.assert_array_equal(back, t)
    except ImportError:
        pass


def test_argument_validation_of_the_widened_entry_points(lib):
    """Error codes of the wider entry points, also returned before any device work."""
    import ctypes as c
    buf = np.zeros(8192, dtype=np.uint8)
    p = (buf.ctypes.data + 255) & ~255
    vp, i, f32 = c.c_void_p, c.c_int, c.c_float

    def sig(fn, types):
        fn.restype, fn.argtypes = c.c_int, types
        return fn

    gqa = sig(lib.sigattn_fwd_gqa, [vp] * 4 + [i] * 5 + [f32, f32, vp, i, vp, i, vp])
    assert gqa(p, p, p, p, 1, 6, 4, 4, 64, 0.125, 0.0, None, 0, None, 0, None) == -2      # H not a multiple of H_kv
    assert gqa(p, p, p, p, 1, 6, 0, 4, 64, 0.125, 0.0, None, 0, None, 0, None) == -2
    assert gqa(p, p, p, p, 1, 6, 3, 4, 64, 0.125, 0.0, p + 2, 0, None, 0, None) == -3     # bias vector alignment
    nk = sig(lib.sigattn_fwd_nk, [vp] * 4 + [i] * 6 + [f32, f32, vp, i, vp, i, vp])
    assert nk(p, p, p, p, 1, 2, 2, 8, 4, 64, 0.125, 0.0, None, 1, None, 0, None) == -2    # causal needs N_k >= N_q
    assert nk(p, p, None, p, 1, 2, 2, 4, 8, 64, 0.125, 0.0, None, 1, None, 0, None) == -1
    shard = sig(lib.sigattn_fwd_shard, [vp] * 4 + [i] * 6 + [f32, f32, vp, i, i, vp, i, vp])
    assert shard(p, p, p, p, 1, 2, 2, 4, 8, 64, 0.125, 0.0, None, 1, (1 << 30) + 1, None, 0, None) == -2   # pos0 out of range
    varlen = sig(lib.sigattn_fwd_varlen, [vp] * 4 + [i] * 5 + [f32, f32, vp, i, vp, vp, i, vp])
    assert varlen(p, p, p, p, 1, 2, 2, 4, 64, 0.125, 0.0, None, 0, None, None, 0, None) == -1             # no lengths
    assert varlen(p, p, p, p, 1, 2, 2, 4, 64, 0.125, 0.0, None, 0, p + 2, None, 0, None) == -3
    ragged = sig(lib.sigattn_fwd_ragged, [vp] * 4 + [i] * 4 + [vp, i, f32, f32, vp, i, vp, i, vp])
    assert ragged(p, p, p, p, 2, 2, 4, 64, None, 1, 0.125, 0.0, None, 0, None, 0, None) == -1
    assert ragged(p, p, p, p, 2, 2, 4, 64, p, 0, 0.125, 0.0, None, 0, None, 0, None) == -2                # no sequences
    rows = sig(lib.sigattn_fwd_rowscale, [vp] * 4 + [i] * 6 + [f32, f32, vp, i, vp, vp, i, vp])
    assert rows(p, p, p, p, 1, 2, 2, 4, 4, 64, 0.125, 0.0, None, 0, None, None, 0, None) == -1            # no factors
    norm = sig(lib.sigattn_seqlen_norm, [vp, i, i, f32, i, vp])
    assert norm(None, 4, 4, 0.5, 1, None) == -1
    assert norm(p, 8, 4, 0.5, 1, None) == -2                                                              # causal needs N_k >= N_q
    assert norm(p, 4, 4, 0.5, 3, None) == -4
    dec = sig(lib.sigattn_fwd_decode, [vp] * 4 + [i] * 6 + [f32, f32, vp, i, vp, i, vp, c.c_size_t, vp])
    assert dec(p, p, p, p, 1, 2, 2, 1, 8, 64, 0.125, 0.0, None, 1, None, 0, None, 0, None) == -1          # workspace missing
    assert dec(p, p, p, p, 1, 2, 2, 1, 8, 64, 0.125, 0.0, None, 1, None, 0, p, 16, None) == -5
    lib.sigattn_fwd_decode_workspace_bytes.restype = c.c_size_t
    lib.sigattn_fwd_decode_workspace_bytes.argtypes = [i] * 5
    assert lib.sigattn_fwd_decode_workspace_bytes(2, 4, 3, 128, 0) == 2 * 4 * 3 * 128 * 4
    assert lib.sigattn_fwd_decode_workspace_bytes(2, 4, 3, 128, 1) == 0
    acc = sig(lib.sigattn_fwd_shard_acc, [vp] * 4 + [i] * 6 + [f32, f32, vp, i, i, vp, i, vp])
    assert acc(p, p, p, None, 1, 2, 2, 4, 8, 64, 0.125, 0.0, None, 1, 0, None, 0, None) == -1             # no accumulator
    assert acc(p, p, p, p, 1, 2, 2, 4, 8, 64, 0.125, 0.0, None, 1, 0, None, 1, None) == -4                # bf16 only
    conv = sig(lib.sigattn_acc_to_bf16, [vp, vp, c.c_size_t, f32, vp])
    assert conv(p, None, 8, 1.0, None) == -1
    assert conv(p, p, 6, 1.0, None) == -2                                                                 # n not a multiple of 4


def test_binding_refuses_slopes_and_workspaces_the_kernels_could_not_read():
    """The Python wrappers check slopes (float32, CUDA, q's device, one per head) and scratch tensors
    (uint8, CUDA, q's device) before any launch: a CPU, float64 or short tensor would make a kernel read
    a host address or past the end, which on a GPU is a fault, not an exception."""
    import torch
    from paper_2409_04431_b200 import binding
    q = torch.zeros(1, 4, 8, 64)
    for bad in (torch.ones(4), torch.ones(4, dtype=torch.float64), torch.ones(3), [0.5] * 4, np.ones(4, np.float32)):
        with pytest.raises(ValueError):
            binding._slopes_ptr(bad, q)       # not on a GPU (and wrong dtype, length or type)
    assert binding._slopes_ptr(None, q) is None
    with pytest.raises(ValueError):
        binding._ws_ptr(torch.zeros(64, dtype=torch.uint8), q)   # host memory
    assert binding._ws_ptr(None, q) is None
    # sigattn_step_host is the one entry point that takes the slopes from the host
    ok = torch.ones(4)
    assert binding._host_slopes_ptr(ok, 4) == ok.data_ptr()
    for bad in (torch.ones(4, dtype=torch.float64), torch.ones(5), torch.ones(8)[::2]):
        with pytest.raises(ValueError):
            binding._host_slopes_ptr(bad, 4)


def test_host_side_check_of_row_offsets(lib):
    import ctypes as c
    lib.sigattn_check_cu_seqlens.restype, lib.sigattn_check_cu_seqlens.argtypes = c.c_int, [c.c_void_p, c.c_int, c.c_int]
    ok = np.array([0, 3, 3, 10], dtype=np.int32)
    assert lib.sigattn_check_cu_seqlens(ok.ctypes.data, 3, 10) == 0
    assert lib.sigattn_check_cu_seqlens(ok.ctypes.data, 3, 11) == -2                      # does not end at T
    assert lib.sigattn_check_cu_seqlens(np.array([1, 3, 10], np.int32).ctypes.data, 2, 10) == -2   # does not start at 0
    assert lib.sigattn_check_cu_seqlens(np.array([0, 7, 5, 10], np.int32).ctypes.data, 3, 10) == -2   # decreases
    assert lib.sigattn_check_cu_seqlens(None, 3, 10) == -1
    import torch
    from paper_2409_04431_b200 import binding
    binding.sigattn_check_cu_seqlens(torch.tensor([0, 4, 9], dtype=torch.int32), 9)
    with pytest.raises(binding.SigattnError):
        binding.sigattn_check_cu_seqlens(torch.tensor([0, 9, 4, 9], dtype=torch.int32), 9)
