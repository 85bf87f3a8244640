"""Gradient of the learnable temperature (sigattn_bwd_dtemp) against the float64 oracle, through the
C ABI: bf16 tensor-core path at the bf16 tolerance, fp32 debug path at 1e-5; the other gradients the
call returns must be those of sigattn_bwd bit for bit (dQ to tolerance: its accumulation order varies)."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, FP32_REL, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,N,D,causal,with_slopes", [
    (2, 3, 300, 64, True, True),      # ragged tiles, position bias
    (1, 4, 1024, 128, True, False),   # several key tiles per head
    (2, 2, 197, 64, False, False),    # no mask
    (1, 2, 1, 128, True, False),      # one token
])
def test_temperature_gradient_bf16(B, H, N, D, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = inputs.random_case(B, H, N, D, seed=7100 + N + D)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    t = 0.25
    scale, bias = math.exp(t) / math.sqrt(D), -math.log(max(N, 2))
    tq, tk, tv, tdo = (to_device(x, "bf16") for x in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    dq, dk, dv, dtemp, dbias = sa.sigattn_bwd_dtemp(tq, tk, tv, tdo, scale, bias, causal, sl)
    sa.sigattn_check()
    assert dbias is None and dtemp.shape == (B, H)
    ref = oracle.sigattn_bwd_dtemp(q, k, v, d_o, scale, bias, causal, slopes)
    got = dtemp.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    # one scalar per head is a sum with cancelling terms: judged over all heads together, like db
    assert rel_fro(got, ref) < BF16_REL_FRO, (got, ref)
    plain = sa.sigattn_bwd(tq, tk, tv, tdo, scale, bias, causal, sl)
    sa.sigattn_check()
    assert torch.equal(dk, plain[1]) and torch.equal(dv, plain[2])
    assert rel_fro(to_host(dq), to_host(plain[0])) < 1e-3


def test_temperature_gradient_with_bias_vector_and_bias_gradient():
    import torch
    import paper_2409_04431_b200 as sa
    B, H, N, D = 2, 4, 640, 128
    q, k, v, d_o = inputs.random_case(B, H, N, D, seed=7200)
    bias = (-math.log(N) + 0.3 * np.random.default_rng(7201).standard_normal((B, H))).astype(np.float32)
    scale = 1.1 / math.sqrt(D)
    tq, tk, tv, tdo = (to_device(x, "bf16") for x in (q, k, v, d_o))
    out = sa.sigattn_bwd_dtemp(tq, tk, tv, tdo, scale, torch.from_numpy(bias).cuda(), True, None, want_dbias=True)
    sa.sigattn_check()
    ref_t = oracle.sigattn_bwd_dtemp(q, k, v, d_o, scale, bias.astype(np.float64), True)
    ref_b = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias.astype(np.float64), True)
    assert rel_fro(out[3].double().cpu().numpy(), ref_t) < BF16_REL_FRO
    assert rel_fro(out[4].double().cpu().numpy(), ref_b) < BF16_REL_FRO


def test_temperature_gradient_fp32_path():
    import paper_2409_04431_b200 as sa
    B, H, N, D = 1, 2, 150, 64
    q, k, v, d_o = inputs.random_case(B, H, N, D, seed=7300, dtype="fp32")
    tq, tk, tv, tdo = (to_device(x, "fp32") for x in (q, k, v, d_o))
    scale, bias = 0.9 / math.sqrt(D), -math.log(N)
    out = sa.sigattn_bwd_dtemp(tq, tk, tv, tdo, scale, bias, True)
    sa.sigattn_check()
    ref = oracle.sigattn_bwd_dtemp(q, k, v, d_o, scale, bias, True)
    assert rel_fro(out[3].double().cpu().numpy(), ref) < FP32_REL
