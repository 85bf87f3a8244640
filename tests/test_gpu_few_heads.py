"""One long causal sequence with few heads: the forward divides the key tiles of every work item
over several items that add their shares of O, the backward with grouped heads divides a group's
query heads.  Parity against the float64 oracle, through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


def test_forward_without_mask_few_items():
    """No mask, 34 work items of 33 key tiles each: divided in two."""
    import paper_2409_04431_b200 as sa
    B, H, N, D = 1, 2, 4224, 64
    q, k, v, _ = inputs.random_case(B, H, N, D, 251)
    tq, tk, tv = (to_device(t, "bf16") for t in (q, k, v))
    scale, bias = 1.0 / math.sqrt(D), -math.log(N)
    o = sa.sigattn_fwd(tq, tk, tv, scale, bias, False)
    sa.sigattn_check()
    ref = oracle.sigattn_fwd(q, k, v, scale, bias, False)
    assert rel_fro(to_host(o), ref) < BF16_REL_FRO
    assert max_abs(to_host(o), ref) < 2e-2 * max(1.0, float(np.abs(ref).max()))


@pytest.mark.parametrize("B,H,N,D,with_slopes", [
    (1, 2, 4224, 128, False),     # 33 key tiles, 34 work items: two parts per item
    (1, 3, 4300, 64, True),       # ragged tail, ALiBi
    (2, 4, 4100, 128, False),     # 136 items: two parts, the short items are not cut
    (1, 24, 4100, 64, False),     # 408 items: enough, no split (same entry point, other path)
])
def test_forward_with_split_key_tiles(B, H, N, D, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, _ = inputs.random_case(B, H, N, D, 221)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv = (to_device(t, "bf16") for t in (q, k, v))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale, bias = 1.0 / math.sqrt(D), -math.log(N)
    o = sa.sigattn_fwd(tq, tk, tv, scale, bias, True, sl)
    sa.sigattn_check()
    ref = oracle.sigattn_fwd(q, k, v, scale, bias, True, slopes)
    g = to_host(o)
    assert np.isfinite(g).all()
    assert rel_fro(g, ref) < BF16_REL_FRO, rel_fro(g, ref)
    assert max_abs(g, ref) < 2e-2 * max(1.0, float(np.abs(ref).max()))
    o2 = sa.sigattn_fwd(tq, tk, tv, scale, bias, True, sl)
    assert torch.equal(o2, o)       # two parts: their sum does not depend on the order of arrival


def test_forward_split_with_query_offset_and_row_factors():
    import torch
    import paper_2409_04431_b200 as sa
    B, H, N_q, N_k, D = 1, 2, 4200, 4500, 128
    q, _, _, _ = inputs.random_case(B, H, N_q, D, 231)
    _, k, v, _ = inputs.random_case(B, H, N_k, D, 232)
    tq, tk, tv = (to_device(t, "bf16") for t in (q, k, v))
    scale, bias = 1.0 / math.sqrt(D), -math.log(N_k)
    o = sa.sigattn_fwd_nk(tq, tk, tv, scale, bias, True)
    ref = oracle.sigattn_fwd(q, k, v, scale, bias, True)
    assert rel_fro(to_host(o), ref) < BF16_REL_FRO
    r = sa.sigattn_seqlen_norm(N_q, N_k, 0.5, True, "cuda")
    o = sa.sigattn_fwd_rowscale(tq, tk, tv, scale, 0.0, r, True)
    sa.sigattn_check()
    ref = oracle.sigattn_fwd(q, k, v, scale, 0.0, True, row_scale=r.cpu().numpy().astype(np.float64))
    assert rel_fro(to_host(o), ref) < BF16_REL_FRO


def test_backward_multi_query_small_batch():
    """Sixteen query heads on one key/value head, B = 1: the group is divided over work items
    that add their dK, dV."""
    import torch
    import paper_2409_04431_b200 as sa
    B, H, H_kv, N, D = 1, 16, 1, 700, 128
    q, _, _, d_o = inputs.random_case(B, H, N, D, 241)
    _, k, v, _ = inputs.random_case(B, H_kv, N, D, 242)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    scale, bias = 1.0 / math.sqrt(D), -math.log(N)
    dq, dk, dv, db = sa.sigattn_bwd_gqa(tq, tk, tv, tdo, scale, bias, True, want_dbias=True)
    sa.sigattn_check()
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, True)
    for name, g, r in zip(("dQ", "dK", "dV"), (dq, dk, dv), refs):
        g = to_host(g)
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
    ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, True)
    assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO


@pytest.mark.parametrize("B,H,N,D,causal,with_slopes", [
    (1, 2, 2100, 128, True, False),      # 34 work items: the query tiles of every key tile go to two items
    (1, 3, 1000, 64, False, True),       # no mask, ragged tail, ALiBi
    (1, 1, 2200, 128, True, True),       # one head
])
def test_backward_with_divided_query_tiles(B, H, N, D, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = inputs.random_case(B, H, N, D, 261)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale, bias = 1.0 / math.sqrt(D), -math.log(N)
    g1 = sa.sigattn_bwd(tq, tk, tv, tdo, scale, bias, causal, sl)
    g2 = sa.sigattn_bwd(tq, tk, tv, tdo, scale, bias, causal, sl)
    sa.sigattn_check()
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes)
    for name, g, r in zip(("dQ", "dK", "dV"), g1, refs):
        g = to_host(g)
        assert np.isfinite(g).all(), name
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
    assert torch.equal(g1[1], g2[1]) and torch.equal(g1[2], g2[2])    # two shares: dK, dV stay bit-reproducible
