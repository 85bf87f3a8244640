"""Seeded random sweep over shapes and options of the widest entry points (N_q queries against
N_k keys, grouped heads, bias per head, ALiBi, causal or not), forward and backward against the
float64 oracle.  Catches index arithmetic that the hand-picked cases miss."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


def _draw(case):
    rng = np.random.default_rng(1000 + case)
    D = int(rng.choice([64, 128]))
    H_kv = int(rng.integers(1, 4))
    group = int(rng.integers(1, 4))
    B = int(rng.integers(1, 3))
    causal = bool(rng.integers(0, 2))
    N_q = int(rng.integers(1, 420))
    N_k = int(rng.integers(N_q, 640)) if causal else int(rng.integers(1, 640))
    return dict(B=B, H=H_kv * group, H_kv=H_kv, N_q=N_q, N_k=N_k, D=D, causal=causal,
                with_slopes=bool(rng.integers(0, 2)), bias_vec=bool(rng.integers(0, 2)))


@pytest.mark.parametrize("case", range(16))
def test_random_case(case):
    import torch
    import paper_2409_04431_b200 as sa
    c = _draw(case)
    B, H, H_kv, N_q, N_k, D = c["B"], c["H"], c["H_kv"], c["N_q"], c["N_k"], c["D"]
    q, _, _, d_o = inputs.random_case(B, H, N_q, D, 300 + case)
    _, k, v, _ = inputs.random_case(B, H_kv, N_k, D, 400 + case)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if c["with_slopes"] else None
    scale = 1.0 / math.sqrt(D)
    if c["bias_vec"]:
        bias_np = (-math.log(N_k) + 0.5 * np.random.default_rng(case).standard_normal((B, H))).astype(np.float32)
        tb, b64 = torch.from_numpy(bias_np).cuda(), bias_np.astype(np.float64)
    else:
        tb = b64 = -math.log(N_k)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    o = sa.sigattn_fwd_nk(tq, tk, tv, scale, tb, c["causal"], sl)
    dq, dk, dv, db = sa.sigattn_bwd_nk(tq, tk, tv, tdo, scale, tb, c["causal"], sl, want_dbias=c["bias_vec"])
    sa.sigattn_check()
    ref_o = oracle.sigattn_fwd(q, k, v, scale, b64, c["causal"], slopes)
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, b64, c["causal"], slopes)
    for name, g, r in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), (ref_o,) + tuple(refs)):
        g = to_host(g)
        assert np.isfinite(g).all(), (name, c)
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r), c)
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), (name, c)
    if c["bias_vec"]:
        ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, b64, c["causal"], slopes)
        assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO, c
