"""GPU parity of multi-query / grouped-query attention (k, v with fewer heads than q)
against the float64 oracle, through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


def _case(B, H, H_kv, N, D, seed, dtype="bf16"):
    q, _, _, d_o = inputs.random_case(B, H, N, D, seed, dtype=dtype)
    _, k, v, _ = inputs.random_case(B, H_kv, N, D, seed + 1, dtype=dtype)
    return q, k, v, d_o


@pytest.mark.parametrize("B,H,H_kv,N,D,causal,with_slopes", [
    (2, 4, 1, 300, 64, True, True),      # multi-query, ragged, ALiBi per query head
    (1, 8, 2, 513, 128, True, False),    # groups of four, several tiles, causal
    (2, 6, 3, 200, 128, False, False),   # groups of two, non-causal
    (1, 4, 4, 130, 64, False, True),     # H_kv == H: plain multi-head attention
])
def test_gqa_bf16(B, H, H_kv, N, D, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = _case(B, H, H_kv, N, D, 51)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale, bias = 1.0 / math.sqrt(D), -math.log(N)
    o = sa.sigattn_fwd_gqa(tq, tk, tv, scale, bias, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_gqa(tq, tk, tv, tdo, scale, bias, causal, sl, want_dbias=True)
    sa.sigattn_check()
    assert dk.shape == tk.shape and dv.shape == tv.shape
    ref_o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes)
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes)
    for name, g, r in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), (ref_o,) + tuple(refs)):
        g = to_host(g)
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
    ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes)
    assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO
    if H_kv == H:   # the grouped entry points with one head per group are the plain ones
        assert torch.equal(o, sa.sigattn_fwd(tq, tk, tv, scale, bias, causal, sl))
        plain = sa.sigattn_bwd(tq, tk, tv, tdo, scale, bias, causal, sl)
        assert torch.equal(dk, plain[1]) and torch.equal(dv, plain[2])


def test_gqa_fp32_debug_path_with_bias_vector():
    import torch
    import paper_2409_04431_b200 as sa
    B, H, H_kv, N, D = 2, 4, 2, 80, 64
    q, k, v, d_o = _case(B, H, H_kv, N, D, 61, dtype="fp32")
    bias = (-math.log(N) + 0.1 * np.random.default_rng(62).standard_normal((B, H))).astype(np.float32)
    tq, tk, tv, tdo = (to_device(t, "fp32") for t in (q, k, v, d_o))
    tb = torch.from_numpy(bias).cuda()
    o = sa.sigattn_fwd_gqa(tq, tk, tv, 0.125, tb, True)
    dq, dk, dv, db = sa.sigattn_bwd_gqa(tq, tk, tv, tdo, 0.125, tb, True, want_dbias=True)
    sa.sigattn_check()
    b64 = bias.astype(np.float64)
    assert rel_fro(to_host(o), oracle.sigattn_fwd(q, k, v, 0.125, b64, True)) < 1e-5
    for g, r in zip((dq, dk, dv), oracle.sigattn_bwd(q, k, v, d_o, 0.125, b64, True)):
        assert rel_fro(to_host(g), r) < 1e-5
    assert rel_fro(db.cpu().numpy().astype(np.float64), oracle.sigattn_bwd_dbias(q, k, v, d_o, 0.125, b64, True)) < 1e-5


def test_gqa_rejects_bad_head_counts():
    import torch
    import paper_2409_04431_b200 as sa
    q = torch.zeros(1, 4, 64, 64, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 3, 64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sa.SigattnError) as e:
        sa.sigattn_fwd_gqa(q, kv, kv, 0.125, -4.0)
    assert e.value.code == -2
