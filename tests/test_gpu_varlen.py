"""GPU parity of padded batches with per-sequence lengths against the float64 oracle,
through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,H_kv,N,D,lens,causal,with_slopes", [
    (4, 2, 2, 300, 64, [300, 171, 128, 1], True, True),       # full, ragged, tile-aligned, one token
    (3, 4, 2, 520, 128, [513, 256, 40], False, False),        # grouped heads, no mask
    (2, 2, 2, 260, 128, [0, 260], True, False),               # an empty sequence
    (2, 3, 1, 700, 64, [699, 385], False, True),              # multi-query with a position bias
])
def test_varlen_bf16(B, H, H_kv, N, D, lens, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, _, _, d_o = inputs.random_case(B, H, N, D, 111)
    _, k, v, _ = inputs.random_case(B, H_kv, N, D, 112)
    # whatever sits in the padding must not matter: make it large
    for b, n in enumerate(lens):
        for t in (q, k, v, d_o):
            t[b, :, n:] = 64.0
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    bias = np.repeat(-np.log(np.maximum(np.array(lens, dtype=np.float64), 1.0))[:, None], H, axis=1).astype(np.float32)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    tb = torch.from_numpy(bias).cuda()
    tl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scale = 1.0 / math.sqrt(D)
    o = sa.sigattn_fwd_varlen(tq, tk, tv, scale, tb, tl, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_varlen(tq, tk, tv, tdo, scale, tb, tl, causal, sl, want_dbias=True)
    sa.sigattn_check()
    b64 = bias.astype(np.float64)
    ref_o = oracle.sigattn_fwd(q, k, v, scale, b64, causal, slopes, seqlens=lens)
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, b64, causal, slopes, seqlens=lens)
    for name, g, r in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), (ref_o,) + tuple(refs)):
        g = to_host(g)
        assert np.isfinite(g).all(), name
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
        for b, n in enumerate(lens):
            assert np.all(g[b, :, n:] == 0.0), (name, b)          # padded rows are exactly zero
    ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, b64, causal, slopes, seqlens=lens)
    assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO


def test_varlen_full_lengths_equal_the_plain_call_and_fp32_path():
    import torch
    import paper_2409_04431_b200 as sa
    B, H, N, D = 2, 2, 200, 64
    q, k, v, d_o = inputs.random_case(B, H, N, D, 121)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    full = torch.full((B,), N, dtype=torch.int32, device="cuda")
    assert torch.equal(sa.sigattn_fwd_varlen(tq, tk, tv, 0.125, -5.0, full, True), sa.sigattn_fwd(tq, tk, tv, 0.125, -5.0, True))
    g = sa.sigattn_bwd_varlen(tq, tk, tv, tdo, 0.125, -5.0, full, True)
    plain = sa.sigattn_bwd(tq, tk, tv, tdo, 0.125, -5.0, True)
    assert torch.equal(g[1], plain[1]) and torch.equal(g[2], plain[2])
    # fp32 debug path
    lens = [150, 7]
    q32, k32, v32, do32 = inputs.random_case(B, H, N, D, 122, dtype="fp32")
    t32 = [to_device(t, "fp32") for t in (q32, k32, v32, do32)]
    tl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    o = sa.sigattn_fwd_varlen(t32[0], t32[1], t32[2], 0.125, -4.0, tl, True)
    dq, dk, dv, db = sa.sigattn_bwd_varlen(*t32, 0.125, -4.0, tl, True, want_dbias=True)
    sa.sigattn_check()
    assert rel_fro(to_host(o), oracle.sigattn_fwd(q32, k32, v32, 0.125, -4.0, True, seqlens=lens)) < 1e-5
    for got, r in zip((dq, dk, dv), oracle.sigattn_bwd(q32, k32, v32, do32, 0.125, -4.0, True, seqlens=lens)):
        assert rel_fro(to_host(got), r) < 1e-5
    assert rel_fro(db.cpu().numpy().astype(np.float64),
                   oracle.sigattn_bwd_dbias(q32, k32, v32, do32, 0.125, -4.0, True, seqlens=lens)) < 1e-5
