"""GPU parity of the cache-decoding forward with keys split over thread blocks against the
float64 oracle, through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,H_kv,N_q,N_k,D,causal,with_slopes", [
    (1, 2, 2, 1, 3000, 128, True, False),      # one token, plain heads: 2 items, keys split many ways
    (2, 8, 2, 1, 2049, 128, True, True),       # grouped heads packed and split, ragged last key tile
    (1, 4, 1, 3, 1500, 64, True, True),        # multi-query, three new tokens: the mask cuts the last split
    (1, 2, 2, 5, 700, 64, False, False),       # no mask (cross-attention against a long memory)
    (3, 4, 4, 128, 1100, 128, True, False),    # a full tile of queries per head
    (1, 1, 1, 1, 100, 64, True, False),        # one key tile: nothing to split
])
def test_decode_split_keys_bf16(B, H, H_kv, N_q, N_k, D, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, _, _, _ = inputs.random_case(B, H, N_q, D, 171)
    _, k, v, _ = inputs.random_case(B, H_kv, N_k, D, 172)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    bias = (-math.log(N_k) + 0.3 * np.random.default_rng(173).standard_normal((B, H))).astype(np.float32)
    tq, tk, tv = (to_device(t, "bf16") for t in (q, k, v))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale = 1.0 / math.sqrt(D)
    tb = torch.from_numpy(bias).cuda()
    o = sa.sigattn_fwd_decode(tq, tk, tv, scale, tb, causal, sl)
    sa.sigattn_check()
    ref = oracle.sigattn_fwd(q, k, v, scale, bias.astype(np.float64), causal, slopes)
    g = to_host(o)
    assert np.isfinite(g).all()
    assert rel_fro(g, ref) < BF16_REL_FRO, rel_fro(g, ref)
    assert max_abs(g, ref) < 2e-2 * max(1.0, float(np.abs(ref).max()))
    # the unsplit entry point agrees to the rounding of the result (fp32 partial sums differ in order)
    o_nk = to_host(sa.sigattn_fwd_nk(tq, tk, tv, scale, tb, causal, sl))
    assert max_abs(g, o_nk) <= 2.0 ** -7 * max(1.0, float(np.abs(o_nk).max()))


def test_decode_many_queries_is_the_plain_path_and_workspace_is_checked():
    import torch
    import paper_2409_04431_b200 as sa
    B, H, N_q, N_k, D = 1, 2, 300, 600, 64
    q, _, _, _ = inputs.random_case(B, H, N_q, D, 181)
    _, k, v, _ = inputs.random_case(B, H, N_k, D, 182)
    tq, tk, tv = (to_device(t, "bf16") for t in (q, k, v))
    scale = 1.0 / math.sqrt(D)
    ws = torch.full((sa.sigattn_fwd_decode_workspace_bytes(B, H, N_q, D, 0),), 7, dtype=torch.uint8, device="cuda")
    o = sa.sigattn_fwd_decode(tq, tk, tv, scale, -2.0, True, workspace=ws)
    # the same kernels either way; the call without scratch may divide its few work items over the keys
    # and add bf16 shares, so the two agree to single roundings
    assert rel_fro(to_host(o), to_host(sa.sigattn_fwd_nk(tq, tk, tv, scale, -2.0, True)).astype(np.float64)) < 4e-3
    assert bool((ws == 7).all())                          # more than one pair of query tiles: no split, no scratch use
    with pytest.raises(sa.SigattnError) as e:
        sa.sigattn_fwd_decode(tq, tk, tv, scale, -2.0, True, workspace=ws[:-256])
    assert e.value.code == -5


@pytest.mark.parametrize("B,H,H_kv,N_k", [
    (8, 32, 32, 16384),      # the measured plain-head decode case
    (1, 32, 8, 131072),      # the measured long-cache grouped-head case (8 work items unsplit)
])
def test_decode_full_size_cases(B, H, H_kv, N_k):
    """The decode cases whose times are reported, checked in full against the oracle (one query
    per head keeps the float64 reference cheap)."""
    import torch
    import paper_2409_04431_b200 as sa
    D = 128
    q, _, _, _ = inputs.random_case(B, H, 1, D, 191)
    _, k, v, _ = inputs.random_case(B, H_kv, N_k, D, 192)
    tq, tk, tv = (to_device(t, "bf16") for t in (q, k, v))
    scale, bias = 1.0 / math.sqrt(D), -math.log(N_k)
    o = sa.sigattn_fwd_decode(tq, tk, tv, scale, bias, True)
    sa.sigattn_check()
    ref = oracle.sigattn_fwd(q, k, v, scale, bias, True)
    g = to_host(o)
    assert np.isfinite(g).all()
    assert rel_fro(g, ref) < BF16_REL_FRO, rel_fro(g, ref)
    assert max_abs(g, ref) < 2e-2 * max(1.0, float(np.abs(ref).max()))
