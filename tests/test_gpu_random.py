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


@pytest.mark.parametrize("case", range(10))
def test_random_batches_of_different_lengths(case):
    """The same random batch of sequences through the padded entry points and through the ones
    without padding, both against the oracle."""
    import torch
    import paper_2409_04431_b200 as sa
    rng = np.random.default_rng(2000 + case)
    D = int(rng.choice([64, 128]))
    H_kv = int(rng.integers(1, 3))
    H = H_kv * int(rng.integers(1, 3))
    n_seqs = int(rng.integers(1, 7))
    lens = [int(x) for x in rng.integers(0 if n_seqs > 1 else 1, 330, size=n_seqs)]
    if sum(lens) == 0:
        lens[0] = 5
    causal = bool(rng.integers(0, 2))
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if rng.integers(0, 2) else None
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale = 1.0 / math.sqrt(D)
    bias = (-np.log(np.maximum(np.array(lens, dtype=np.float64), 1.0))[:, None] + 0.2 * rng.standard_normal((n_seqs, H))).astype(np.float32)
    tb = torch.from_numpy(bias).cuda()
    b64 = bias.astype(np.float64)
    tag = dict(case=case, D=D, H=H, H_kv=H_kv, lens=lens, causal=causal, slopes=slopes is not None)

    def check(outs, refs, ref_db, db):
        for name, g, r in zip(("O", "dQ", "dK", "dV"), outs, refs):
            g = to_host(g)
            assert np.isfinite(g).all(), (name, tag)
            assert rel_fro(g, r) < BF16_REL_FRO, (name, rel_fro(g, r), tag)
            assert max_abs(g, r) < 2e-2 * max(1.0, float(np.abs(r).max())), (name, tag)
        assert rel_fro(db.cpu().numpy().astype(np.float64), ref_db) < BF16_REL_FRO, tag

    # without padding
    T = sum(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q, _, _, d_o = inputs.random_case(1, H, T, D, 500 + case)
    _, k, v, _ = inputs.random_case(1, H_kv, T, D, 600 + case)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    tcu = torch.from_numpy(cu).cuda()
    o = sa.sigattn_fwd_ragged(tq, tk, tv, tcu, scale, tb, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_ragged(tq, tk, tv, tdo, tcu, scale, tb, causal, sl, want_dbias=True)
    sa.sigattn_check()
    check((o, dq, dk, dv),
          (oracle.sigattn_fwd(q, k, v, scale, b64, causal, slopes, cu_seqlens=cu),) + tuple(
              oracle.sigattn_bwd(q, k, v, d_o, scale, b64, causal, slopes, cu_seqlens=cu)),
          oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, b64, causal, slopes, cu_seqlens=cu), db)

    # padded to the longest sequence (rounded up a little so that some padding always exists)
    N = max(lens) + int(rng.integers(1, 40))
    qp, _, _, dop = inputs.random_case(n_seqs, H, N, D, 700 + case)
    _, kp, vp, _ = inputs.random_case(n_seqs, H_kv, N, D, 800 + case)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (qp, kp, vp, dop))
    tl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    o = sa.sigattn_fwd_varlen(tq, tk, tv, scale, tb, tl, causal, sl)
    dq, dk, dv, db = sa.sigattn_bwd_varlen(tq, tk, tv, tdo, scale, tb, tl, causal, sl, want_dbias=True)
    sa.sigattn_check()
    check((o, dq, dk, dv),
          (oracle.sigattn_fwd(qp, kp, vp, scale, b64, causal, slopes, seqlens=lens),) + tuple(
              oracle.sigattn_bwd(qp, kp, vp, dop, scale, b64, causal, slopes, seqlens=lens)),
          oracle.sigattn_bwd_dbias(qp, kp, vp, dop, scale, b64, causal, slopes, seqlens=lens), db)


@pytest.mark.parametrize("case", range(8))
def test_random_decode_and_row_factors(case):
    """Random cache-decoding shapes through the split-key forward, and random row factors through
    forward and backward."""
    import torch
    import paper_2409_04431_b200 as sa
    rng = np.random.default_rng(3000 + case)
    D = int(rng.choice([64, 128]))
    H_kv = int(rng.integers(1, 4))
    H = H_kv * int(rng.integers(1, 5))
    B = int(rng.integers(1, 3))
    N_q = int(rng.integers(1, 9))
    N_k = int(rng.integers(max(N_q, 130), 5000))
    causal = bool(rng.integers(0, 2))
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if rng.integers(0, 2) else None
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale, bias = 1.0 / math.sqrt(D), -math.log(N_k)
    tag = dict(case=case, B=B, H=H, H_kv=H_kv, N_q=N_q, N_k=N_k, D=D, causal=causal, slopes=slopes is not None)
    q, _, _, d_o = inputs.random_case(B, H, N_q, D, 900 + case)
    _, k, v, _ = inputs.random_case(B, H_kv, N_k, D, 950 + case)
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    o = sa.sigattn_fwd_decode(tq, tk, tv, scale, bias, causal, sl)
    sa.sigattn_check()
    ref = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes)
    g = to_host(o)
    assert rel_fro(g, ref) < BF16_REL_FRO, (rel_fro(g, ref), tag)
    assert max_abs(g, ref) < 2e-2 * max(1.0, float(np.abs(ref).max())), tag

    r = rng.uniform(0.05, 1.5, size=N_q).astype(np.float32)
    tr = torch.from_numpy(r).cuda()
    o = sa.sigattn_fwd_rowscale(tq, tk, tv, scale, bias, tr, causal, sl)
    dq, dk, dv, _ = sa.sigattn_bwd_rowscale(tq, tk, tv, tdo, scale, bias, tr, causal, sl)
    sa.sigattn_check()
    r64 = r.astype(np.float64)
    refs = (oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes, row_scale=r64),) + tuple(
        oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes, row_scale=r64))
    for name, g, rf in zip(("O", "dQ", "dK", "dV"), (o, dq, dk, dv), refs):
        g = to_host(g)
        assert rel_fro(g, rf) < BF16_REL_FRO, (name, rel_fro(g, rf), tag)
        assert max_abs(g, rf) < 2e-2 * max(1.0, float(np.abs(rf).max())), (name, tag)
