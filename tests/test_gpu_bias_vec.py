"""GPU parity of the bias-vector entry points (one bias per (batch, head), and the bias
gradient db = sum dS) against the float64 oracle, through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


def _bias(B, H, N, seed):
    """Per-sample b = -log n_b for sample lengths n_b <= N, plus a small per-head offset
    as a learnable bias would have."""
    rng = np.random.default_rng(seed)
    n_b = rng.integers(max(1, N // 2), N + 1, size=B)
    return (-np.log(n_b)[:, None] + 0.2 * rng.standard_normal((B, H))).astype(np.float32)


@pytest.mark.parametrize("B,H,N,D,causal,with_slopes", [
    (2, 3, 300, 64, True, True),
    (3, 2, 257, 128, False, False),
    (1, 4, 1000, 128, True, False),
    (2, 2, 64, 64, False, True),
])
def test_bias_vec_bf16(B, H, N, D, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = inputs.random_case(B, H, N, D, seed=31)
    bias = _bias(B, H, N, 32)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    tb = torch.from_numpy(bias).cuda()
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale = 1.0 / math.sqrt(D)
    o = sa.sigattn_fwd_bias_vec(tq, tk, tv, scale, tb, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_bias_vec(tq, tk, tv, tdo, scale, tb, causal, sl)
    sa.sigattn_check()
    ref_o = oracle.sigattn_fwd(q, k, v, scale, bias.astype(np.float64), causal, slopes)
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, bias.astype(np.float64), causal, slopes)
    ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias.astype(np.float64), causal, slopes)
    for name, g, r in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), (ref_o,) + tuple(refs)):
        g = to_host(g)
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
    # the bias gradient is a sum of N^2 signed terms per head: compare all heads together
    got_db = db.cpu().numpy().astype(np.float64)
    assert rel_fro(got_db, ref_db) < BF16_REL_FRO, rel_fro(got_db, ref_db)
    # a scalar bias through the vector entry points equals the scalar entry points bit for bit
    tb1 = torch.full((B, H), -math.log(N), dtype=torch.float32, device="cuda")
    o_vec = sa.sigattn_fwd_bias_vec(tq, tk, tv, scale, tb1, causal, sl)
    o_sc = sa.sigattn_fwd(tq, tk, tv, scale, float(np.float32(-math.log(N))), causal, sl)
    assert torch.equal(o_vec, o_sc)
    g_vec = sa.sigattn_bwd_bias_vec(tq, tk, tv, tdo, scale, tb1, causal, sl, want_dbias=False)
    g_sc = sa.sigattn_bwd(tq, tk, tv, tdo, scale, float(np.float32(-math.log(N))), causal, sl)
    assert g_vec[3] is None
    for a, b in zip(g_vec[1:3], g_sc[1:3]):   # dK, dV: no atomics involved
        assert torch.equal(a, b)


def test_bias_vec_fp32_debug_path():
    import torch
    import paper_2409_04431_b200 as sa
    B, H, N, D = 2, 2, 96, 64
    q, k, v, d_o = inputs.random_case(B, H, N, D, seed=41, dtype="fp32")
    bias = _bias(B, H, N, 42)
    tq, tk, tv, tdo = (to_device(t, "fp32") for t in (q, k, v, d_o))
    tb = torch.from_numpy(bias).cuda()
    o = sa.sigattn_fwd_bias_vec(tq, tk, tv, 0.125, tb, True)
    dq, dk, dv, db = sa.sigattn_bwd_bias_vec(tq, tk, tv, tdo, 0.125, tb, True)
    sa.sigattn_check()
    b64 = bias.astype(np.float64)
    assert rel_fro(to_host(o), oracle.sigattn_fwd(q, k, v, 0.125, b64, True)) < 1e-5
    for g, r in zip((dq, dk, dv), oracle.sigattn_bwd(q, k, v, d_o, 0.125, b64, True)):
        assert rel_fro(to_host(g), r) < 1e-5
    assert rel_fro(db.cpu().numpy().astype(np.float64), oracle.sigattn_bwd_dbias(q, k, v, d_o, 0.125, b64, True)) < 1e-5


def test_bias_vec_argument_errors():
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = (to_device(t, "bf16") for t in inputs.random_case(1, 2, 64, 64, seed=3))
    lib = sa.lib()
    o = torch.empty_like(q)
    args = [q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), 1, 2, 64, 64, 0.125]
    assert lib.sigattn_fwd_bias_vec(*args, None, 0, None, 0, None) == -1          # null bias vector
    tb = torch.zeros(3, dtype=torch.float32, device="cuda")
    assert lib.sigattn_fwd_bias_vec(*args, tb.data_ptr() + 2, 0, None, 0, None) == -3   # misaligned
    with pytest.raises(ValueError):
        sa.sigattn_fwd_bias_vec(q, k, v, 0.125, torch.zeros(2, 1, device="cuda"))
