"""sigattn_bwd_static_scratch: the backward for callers that cannot allocate device memory
(allocator callbacks, real-time loops, plugins whose host forbids allocation after start-up):
they have no workspace to give sigattn_bwd, so the library keeps the fp32 dQ accumulator in a
fixed built-in array.  The entry point must give the same gradients as sigattn_bwd (and meet
the float64 oracle at the usual tolerance), also on a second call that finds the array dirty
from the first, must refuse problems that do not fit the array, and must leave the amount of
free device memory and the caching allocator's counters exactly as it found them.  This file
is named to be collected last."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_MAX_ABS, BF16_REL_FRO, max_abs, rel_fro, to_device, to_host


def test_rejects_problems_beyond_the_built_in_scratch_without_a_gpu():
    from paper_2409_04431_b200 import build
    build.build()
    from paper_2409_04431_b200 import binding
    lib = binding.lib()
    limit = lib.sigattn_bwd_static_scratch_max_elements()
    assert limit == 4 << 20
    buf = np.zeros(4096, dtype=np.uint8)
    p = (buf.ctypes.data + 255) & ~255
    # 1 * 9 * 4096 * 128 elements > 4 Mi: refused before any device work, with its own code and text
    rc = lib.sigattn_bwd_static_scratch(p, p, p, p, p, p, p, 1, 9, 4096, 128, 0.1, 0.0, 1, None, 0, None)
    assert rc == -9
    assert "built-in scratch" in lib.sigattn_strerror(rc).decode()
    assert lib.sigattn_bwd_static_scratch(p, p, p, p, p, p, None, 1, 1, 64, 64, 0.1, 0.0, 1, None, 0, None) == -1
    assert lib.sigattn_bwd_static_scratch(p, p, p, p, p, p, p, 1, 1, 64, 96, 0.1, 0.0, 1, None, 0, None) == -2


@pytest.mark.gpu
def test_static_scratch_backward_matches_workspace_backward_twice_in_a_row():
    import torch
    import paper_2409_04431_b200 as sa

    D = 128
    slopes = torch.tensor([0.5, 0.125, 0.03125], dtype=torch.float32, device="cuda")
    # two different problems back to back: the second call finds the array dirty and smaller/larger than before
    cases = [(2, 3, 600, True, slopes), (1, 3, 1100, False, None)]
    for B, H, N, causal, sl in cases:
        q, k, v, d_o = inputs.random_case(B, H, N, D, seed=4242 + N)
        tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
        scale, bias = 1 / math.sqrt(D), -math.log(N)
        ref = sa.sigattn_bwd(tq, tk, tv, tdo, scale, bias, causal, sl)
        ref64 = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, None if sl is None else sl.cpu().numpy())
        out = tuple(torch.full_like(tq, float("nan")) for _ in range(3))
        for call in range(2):
            # the promise in the name: with the outputs preallocated, the call takes no device memory,
            # neither from the driver (free bytes) nor from torch's caching allocator (its counters)
            torch.cuda.synchronize()
            free0 = torch.cuda.mem_get_info()[0]
            stats0 = torch.cuda.memory_stats()
            got = sa.sigattn_bwd_static_scratch(tq, tk, tv, tdo, scale, bias, causal, sl, out=out)
            sa.sigattn_check()
            stats1 = torch.cuda.memory_stats()
            if call > 0:   # (the very first call on a device may load the module that holds the array)
                assert torch.cuda.mem_get_info()[0] == free0, "free device memory changed across the call"
            for key in ("allocation.all.allocated", "segment.all.allocated", "allocated_bytes.all.allocated"):
                assert stats1[key] == stats0[key], f"caching allocator counter {key} moved"
            for name, g, r in zip(("dQ", "dK", "dV"), got, ref64):
                g64 = to_host(g)
                assert max_abs(g64, r) <= BF16_MAX_ABS, f"{name} call {call} vs oracle"
                assert rel_fro(g64, r) <= BF16_REL_FRO, f"{name} call {call} vs oracle"
            for name, g, r in zip(("dQ", "dK", "dV"), got, ref):
                g64, r64 = to_host(g), to_host(r)
                assert np.all(np.isfinite(g64)), f"{name} call {call}: non-finite"
                assert max_abs(g64, r64) <= BF16_MAX_ABS, f"{name} call {call}"
                assert rel_fro(g64, r64) <= BF16_REL_FRO, f"{name} call {call}"
            # dK and dV do not touch the scratch and are deterministic: bit-identical
            assert torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])

    # fp32 debug path goes through the same entry point (it needs no scratch)
    q, k, v, d_o = inputs.random_case(1, 2, 100, 64, seed=5, dtype="fp32")
    tq, tk, tv, tdo = (to_device(t, "fp32") for t in (q, k, v, d_o))
    ref = sa.sigattn_bwd(tq, tk, tv, tdo, 0.125, -4.0, True)
    got = sa.sigattn_bwd_static_scratch(tq, tk, tv, tdo, 0.125, -4.0, True)
    sa.sigattn_check()
    for g, r in zip(got, ref):
        assert torch.equal(g, r)
