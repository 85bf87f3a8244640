"""Where the bf16 tolerance is tight: a few-token decoding shape with steep ALiBi slopes.

With slopes 2^-1 ... 2^-4 two to five keys carry a query row's whole weight, so a gradient row
is the sum of that many bf16-rounded terms and nothing averages out: the relative Frobenius
error against the float64 oracle sits near (on some seeds above) the 5e-3 that the benchmark
configurations meet with a factor two to spare.  This test pins that the excess is the bf16
arithmetic's, not the kernels': a float64 model of the pipeline that rounds to bf16 exactly
where the kernels do (dO times the row factor, dS, the outputs; P for the forward and dV) and
is exact everywhere else must reproduce the kernels' results ten times more closely than
the oracle does (with one key/value head per query head, so that no partial sums are merged in bf16).  The model is test code: numpy, written from the definition (Section 2, Eq. 3;
Appendix F.1, Algorithm 2 with the 1/sqrt(d) factor), sharing nothing with the CUDA path.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


def _bf16(x):
    return inputs.round_to_bf16(np.asarray(x, dtype=np.float32)).astype(np.float64)


def _model_rowscale_bwd_fwd(q, k, v, d_o, scale, bias, slopes, r):
    """bf16-pipeline model of the causal forward and backward with one factor per query row;
    N_q queries are the last positions of the N_k keys; every query head has its own K, V head."""
    B, H, N_q, D = q.shape
    N_k = k.shape[2]
    pos = np.arange(N_q) + (N_k - N_q)
    keys = np.arange(N_k)
    o = np.zeros((B, H, N_q, D))
    dq = np.zeros((B, H, N_q, D))
    dk = np.zeros((B, H, N_k, D))
    dv = np.zeros((B, H, N_k, D))
    for b in range(B):
        for h in range(H):
            x = scale * (q[b, h] @ k[b, h].T) + bias - slopes[h] * np.abs(pos[:, None] - keys[None, :])
            p = np.where(keys[None, :] > pos[:, None], 0.0, 1.0 / (1.0 + np.exp(-np.clip(x, -700, 700))))
            p16 = _bf16(p)
            o[b, h] = (p16 @ v[b, h]) * r[:, None]
            do_r = _bf16(d_o[b, h] * r[:, None])
            ds = _bf16(p * (1.0 - p) * (do_r @ v[b, h].T))
            dq[b, h] = scale * ds @ k[b, h]
            dk[b, h] += scale * ds.T @ q[b, h]
            dv[b, h] += p16.T @ do_r
    return _bf16(o), _bf16(dq), _bf16(dk), _bf16(dv)


@pytest.mark.parametrize("seed,B,H,N_q,N_k,D", [(240, 1, 4, 4, 3983, 128), (463, 2, 1, 1, 3426, 128),
                                                 (9, 1, 3, 3, 3587, 64), (7, 2, 4, 7, 4131, 128)])
def test_decode_with_steep_slopes_matches_the_bf16_pipeline_model(seed, B, H, N_q, N_k, D):
    import torch
    import paper_2409_04431_b200 as sa
    q, _, _, d_o = inputs.random_case(B, H, N_q, D, 900 + seed)
    _, k, v, _ = inputs.random_case(B, H, N_k, D, 950 + seed)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32)
    r = np.random.default_rng(seed).uniform(0.05, 1.5, size=N_q).astype(np.float32)
    scale, bias = 1.0 / math.sqrt(D), -math.log(N_k)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl, tr = torch.from_numpy(slopes).cuda(), torch.from_numpy(r).cuda()
    o = sa.sigattn_fwd_rowscale(tq, tk, tv, scale, bias, tr, True, sl)
    dq, dk, dv, _ = sa.sigattn_bwd_rowscale(tq, tk, tv, tdo, scale, bias, tr, True, sl)
    sa.sigattn_check()
    r64 = r.astype(np.float64)
    refs = (oracle.sigattn_fwd(q, k, v, scale, bias, True, slopes, row_scale=r64),) + tuple(
        oracle.sigattn_bwd(q, k, v, d_o, scale, bias, True, slopes, row_scale=r64))
    model = _model_rowscale_bwd_fwd(*(t.astype(np.float64) for t in (q, k, v, d_o)), scale, bias,
                                    slopes.astype(np.float64), r64)
    for name, g, rf, m in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), refs, model):
        g = to_host(g)
        assert np.isfinite(g).all(), name
        to_oracle, to_model = rel_fro(g, rf), rel_fro(g, m)
        # bf16 rounding alone bounds the distance to the oracle here (three roundings of at most
        # 2^-9 each on a handful of terms); the kernels must sit on the model, not merely near it
        assert to_oracle < 2e-2, (name, to_oracle)
        # (measured: bit-identical for most outputs, 2e-4 at worst)
        assert to_model < 5e-4, (name, to_model, to_oracle)
