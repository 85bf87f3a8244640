"""GPU parity of N_q queries against N_k keys (queries at the last positions: decoding with
a cache; cross-attention without a mask) against the float64 oracle, through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


def _case(B, H, H_kv, N_q, N_k, D, seed, dtype="bf16"):
    q, _, _, d_o = inputs.random_case(B, H, N_q, D, seed, dtype=dtype)
    _, k, v, _ = inputs.random_case(B, H_kv, N_k, D, seed + 1, dtype=dtype)
    return q, k, v, d_o


@pytest.mark.parametrize("B,H,H_kv,N_q,N_k,D,causal,with_slopes", [
    (2, 4, 4, 1, 1000, 128, True, False),     # one new token against a cache
    (1, 4, 2, 5, 777, 64, True, True),        # a few tokens, grouped heads, ALiBi from the query's position
    (1, 2, 2, 300, 500, 128, True, False),    # offset 200: the mask cuts through two key tiles per query tile
    (2, 2, 1, 256, 384, 64, True, True),      # offset 128: tile-aligned
    (1, 3, 3, 200, 77, 128, False, False),    # cross-attention, fewer keys than queries
    (1, 2, 2, 129, 1025, 64, False, True),    # cross-attention with a position bias
])
def test_nk_bf16(B, H, H_kv, N_q, N_k, D, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = _case(B, H, H_kv, N_q, N_k, D, 71)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale, bias = 1.0 / math.sqrt(D), -math.log(N_k)
    o = sa.sigattn_fwd_nk(tq, tk, tv, scale, bias, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_nk(tq, tk, tv, tdo, scale, bias, causal, sl, want_dbias=True)
    sa.sigattn_check()
    assert o.shape == tq.shape and dq.shape == tq.shape and dk.shape == tk.shape and dv.shape == tv.shape
    ref_o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes)
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes)
    for name, g, r in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), (ref_o,) + tuple(refs)):
        g = to_host(g)
        assert np.isfinite(g).all(), name
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
    ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes)
    assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO


@pytest.mark.parametrize("B,H,H_kv,N_q,N_k,D,causal,with_slopes", [
    (2, 8, 2, 1, 1000, 128, True, False),     # decoding with grouped heads: 4 rows per key/value head
    (1, 8, 1, 3, 500, 64, True, True),        # multi-query, 24 packed rows, slopes per query head
    (1, 4, 1, 64, 300, 128, True, False),     # 256 packed rows: both tiles of one item
    (1, 4, 1, 65, 300, 128, True, False),     # 260 rows: one too many, the unpacked path
    (1, 6, 3, 20, 100, 64, False, True),      # packed, no mask, position bias
])
def test_nk_grouped_heads_packed_forward(B, H, H_kv, N_q, N_k, D, causal, with_slopes):
    """With few queries per head the forward packs the query heads of a key/value head into
    the rows of one tile; each packed row keeps its own head's slope and bias and its own
    position."""
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, _ = _case(B, H, H_kv, N_q, N_k, D, 91)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    bias = (-math.log(N_k) + 0.3 * np.random.default_rng(92).standard_normal((B, H))).astype(np.float32)
    tq, tk, tv = (to_device(t, "bf16") for t in (q, k, v))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale = 1.0 / math.sqrt(D)
    o = sa.sigattn_fwd_nk(tq, tk, tv, scale, torch.from_numpy(bias).cuda(), causal, sl)
    sa.sigattn_check()
    ref = oracle.sigattn_fwd(q, k, v, scale, bias.astype(np.float64), causal, slopes)
    g = to_host(o)
    assert np.isfinite(g).all()
    assert rel_fro(g, ref) < BF16_REL_FRO, rel_fro(g, ref)
    assert max_abs(g, ref) < 2e-2 * max(1.0, float(np.abs(ref).max()))
    # every head on its own (one head per group is never packed) gives the same rows
    for h in range(H):
        hk = h // (H // H_kv)
        one = sa.sigattn_fwd_nk(tq[:, h:h + 1].contiguous(), tk[:, hk:hk + 1].contiguous(), tv[:, hk:hk + 1].contiguous(),
                                scale, torch.from_numpy(bias[:, h:h + 1].copy()).cuda(), causal,
                                None if sl is None else sl[h:h + 1].contiguous())
        assert torch.equal(one, o[:, h:h + 1])


def test_nk_fp32_debug_path():
    import paper_2409_04431_b200 as sa
    B, H, H_kv, N_q, N_k, D = 1, 4, 2, 37, 150, 64
    q, k, v, d_o = _case(B, H, H_kv, N_q, N_k, D, 81, dtype="fp32")
    slopes = np.array([0.5, 0.25, 0.125, 0.0625], dtype=np.float32)
    import torch
    tq, tk, tv, tdo = (to_device(t, "fp32") for t in (q, k, v, d_o))
    sl = torch.from_numpy(slopes).cuda()
    o = sa.sigattn_fwd_nk(tq, tk, tv, 0.125, -5.0, True, sl)
    dq, dk, dv, db = sa.sigattn_bwd_nk(tq, tk, tv, tdo, 0.125, -5.0, True, sl, want_dbias=True)
    sa.sigattn_check()
    assert rel_fro(to_host(o), oracle.sigattn_fwd(q, k, v, 0.125, -5.0, True, slopes)) < 1e-5
    for g, r in zip((dq, dk, dv), oracle.sigattn_bwd(q, k, v, d_o, 0.125, -5.0, True, slopes)):
        assert rel_fro(to_host(g), r) < 1e-5
    assert rel_fro(db.cpu().numpy().astype(np.float64), oracle.sigattn_bwd_dbias(q, k, v, d_o, 0.125, -5.0, True, slopes)) < 1e-5


def test_nk_square_is_the_plain_entry_point_and_causal_needs_enough_keys():
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = (to_device(t, "bf16") for t in inputs.random_case(1, 2, 300, 64, seed=9))
    assert torch.equal(sa.sigattn_fwd_nk(q, k, v, 0.125, -5.0, True), sa.sigattn_fwd(q, k, v, 0.125, -5.0, True))
    with pytest.raises(sa.SigattnError) as e:
        sa.sigattn_fwd_nk(q, k[:, :, :200].contiguous(), v[:, :, :200].contiguous(), 0.125, -5.0, True)
    assert e.value.code == -2
