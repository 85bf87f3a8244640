"""GPU parity of the sequence-length normalisation (one factor per query row, Appendix G
ablation of n^-alpha) against the float64 oracle, through the C ABI."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs
from parity_util import BF16_REL_FRO, max_abs, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_q,n_k,alpha,causal", [(300, 300, 1.0, True), (5, 700, 0.5, True), (260, 100, 0.5, False)])
def test_seqlen_norm_table(n_q, n_k, alpha, causal):
    import paper_2409_04431_b200 as sa
    r = sa.sigattn_seqlen_norm(n_q, n_k, alpha, causal, "cuda").cpu().numpy().astype(np.float64)
    ref = oracle.seqlen_norm(n_q, alpha, causal, n_k=n_k)
    np.testing.assert_allclose(r, ref, rtol=2e-6)


@pytest.mark.parametrize("B,H,H_kv,N_q,N_k,D,alpha,bias,causal,with_slopes", [
    (2, 2, 2, 300, 300, 64, 1.0, 0.0, True, True),         # the paper's causal form, no bias, ALiBi
    (1, 4, 2, 515, 515, 128, 0.5, 0.0, False, False),      # n^-1/2, grouped heads
    (2, 2, 1, 130, 391, 128, 0.5, -2.0, True, False),      # queries at the end of a longer key sequence
    (1, 2, 2, 700, 700, 64, 1.0, None, True, True),        # with a bias per (batch, head) and its gradient
])
def test_rowscale_bf16(B, H, H_kv, N_q, N_k, D, alpha, bias, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, _, _, d_o = inputs.random_case(B, H, N_q, D, 131)
    _, k, v, _ = inputs.random_case(B, H_kv, N_k, D, 132)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale = 1.0 / math.sqrt(D)
    if bias is None:
        bias_np = np.linspace(-3.0, -0.5, B * H).reshape(B, H).astype(np.float32)
        tb, b64 = torch.from_numpy(bias_np).cuda(), bias_np.astype(np.float64)
    else:
        tb, b64 = bias, bias
    tr = sa.sigattn_seqlen_norm(N_q, N_k, alpha, causal, "cuda")
    r64 = tr.cpu().numpy().astype(np.float64)          # the factors the kernels actually read
    o = sa.sigattn_fwd_rowscale(tq, tk, tv, scale, tb, tr, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_rowscale(tq, tk, tv, tdo, scale, tb, tr, causal, sl, want_dbias=True)
    sa.sigattn_check()
    ref_o = oracle.sigattn_fwd(q, k, v, scale, b64, causal, slopes, row_scale=r64)
    refs = oracle.sigattn_bwd(q, k, v, d_o, scale, b64, causal, slopes, row_scale=r64)
    for name, g, r in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), (ref_o,) + tuple(refs)):
        g = to_host(g)
        assert np.isfinite(g).all(), name
        assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r))
        assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), name
    ref_db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, b64, causal, slopes, row_scale=r64)
    assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO


def test_rowscale_fp32_and_unit_factors():
    """fp32 path against the oracle at 1e-5; factors of 1 reproduce the plain call bit for bit."""
    import torch
    import paper_2409_04431_b200 as sa
    B, H, N, D = 1, 2, 150, 64
    q, k, v, d_o = inputs.random_case(B, H, N, D, 141)
    scale, bias = 1.0 / math.sqrt(D), -1.0
    r = np.linspace(0.1, 2.0, N).astype(np.float32)
    tr = torch.from_numpy(r).cuda()
    t32 = [to_device(t, "fp32") for t in (q, k, v, d_o)]
    o = sa.sigattn_fwd_rowscale(*t32[:3], scale, bias, tr, True)
    g = sa.sigattn_bwd_rowscale(*t32, scale, bias, tr, True)[:3]
    sa.sigattn_check()
    r64 = r.astype(np.float64)
    ref = (oracle.sigattn_fwd(q, k, v, scale, bias, True, row_scale=r64),) + tuple(
        oracle.sigattn_bwd(q, k, v, d_o, scale, bias, True, row_scale=r64))
    for name, a, b in zip(("O", "dQ", "dK", "dV"), (o,) + tuple(g), ref):
        assert max_abs(to_host(a), b) < 1e-5 * max(1.0, float(np.abs(b).max())), name
    tb = [to_device(t, "bf16") for t in (q, k, v, d_o)]
    ones = torch.ones(N, dtype=torch.float32, device="cuda")
    assert torch.equal(sa.sigattn_fwd_rowscale(*tb[:3], scale, bias, ones, True), sa.sigattn_fwd(*tb[:3], scale, bias, True))
    for a, b in zip(sa.sigattn_bwd_rowscale(*tb, scale, bias, ones, True)[:3], sa.sigattn_bwd(*tb, scale, bias, True)):
        assert torch.equal(a, b)
    with pytest.raises(ValueError):
        sa.sigattn_fwd_rowscale(*tb[:3], scale, bias, ones[:-1], True)
