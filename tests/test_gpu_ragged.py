"""GPU parity of batches stored without padding (row offsets `cu_seqlens`) against the float64
oracle, through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("H,H_kv,D,lens,causal,with_slopes", [
    (2, 2, 64, [300, 171, 128, 1, 90], True, True),       # boundaries inside tiles, on a tile edge, a single row
    (4, 2, 128, [513, 0, 256, 40], False, False),         # grouped heads, an empty sequence, no mask
    (2, 2, 128, [5, 7, 3, 20, 1, 64, 30, 2], True, False),  # many short sequences inside one tile
    (3, 1, 64, [700, 385], False, True),                  # multi-query with a position bias
    (2, 2, 64, [450], True, False),                       # one sequence: the plain case
])
def test_ragged_bf16(H, H_kv, D, lens, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    T = sum(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q, _, _, d_o = inputs.random_case(1, H, T, D, 201)
    _, k, v, _ = inputs.random_case(1, H_kv, T, D, 202)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    bias = np.repeat(-np.log(np.maximum(np.array(lens, dtype=np.float64), 1.0))[:, None], H, axis=1)
    bias = (bias + 0.1 * np.arange(H)[None, :]).astype(np.float32)                 # one per (sequence, head)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    tb = torch.from_numpy(bias).cuda()
    tcu = torch.from_numpy(cu).cuda()
    scale = 1.0 / math.sqrt(D)
    o = sa.sigattn_fwd_ragged(tq, tk, tv, tcu, scale, tb, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_ragged(tq, tk, tv, tdo, tcu, scale, tb, causal, sl, want_dbias=True)
    sa.sigattn_check()
    b64 = bias.astype(np.float64)
    ref_o = oracle.sigattn_fwd(q, k, v, scale, b64, causal, slopes, cu_seqlens=cu)
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, b64, causal, slopes, cu_seqlens=cu)
    for name, g, r in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), (ref_o,) + tuple(refs)):
        g = to_host(g)
        assert np.isfinite(g).all(), name
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
    ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, b64, causal, slopes, cu_seqlens=cu)
    assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO


def test_ragged_fp32_and_single_sequence_equals_plain_call():
    import torch
    import paper_2409_04431_b200 as sa
    H, D, lens = 2, 64, [70, 130, 9]
    T = sum(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q, k, v, d_o = inputs.random_case(1, H, T, D, 211)
    scale, bias = 1.0 / math.sqrt(D), -2.0
    t32 = [to_device(t, "fp32") for t in (q, k, v, d_o)]
    tcu = torch.from_numpy(cu).cuda()
    o = sa.sigattn_fwd_ragged(*t32[:3], tcu, scale, bias, True)
    g = sa.sigattn_bwd_ragged(*t32, tcu, scale, bias, True)[:3]
    sa.sigattn_check()
    ref = (oracle.sigattn_fwd(q, k, v, scale, bias, True, cu_seqlens=cu),) + tuple(
        oracle.sigattn_bwd(q, k, v, d_o, scale, bias, True, cu_seqlens=cu))
    for name, a, b in zip(("O", "dQ", "dK", "dV"), (o,) + tuple(g), ref):
        assert max_abs(to_host(a), b) < 1e-5 * max(1.0, float(np.abs(b).max())), name
    # one sequence that covers every row is the plain call, bit for bit (dQ up to the order of its atomics)
    tb = [to_device(t, "bf16") for t in (q, k, v, d_o)]
    one = torch.tensor([0, T], dtype=torch.int32, device="cuda")
    assert torch.equal(sa.sigattn_fwd_ragged(*tb[:3], one, scale, bias, True), sa.sigattn_fwd(*tb[:3], scale, bias, True))
    a = sa.sigattn_bwd_ragged(*tb, one, scale, bias, True)
    b = sa.sigattn_bwd(*tb, scale, bias, True)
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    assert max_abs(to_host(a[0]), to_host(b[0]).astype(np.float64)) < 1e-2
    with pytest.raises(ValueError):
        sa.sigattn_fwd_ragged(*tb[:3], one.to(torch.int64), scale, bias, True)
