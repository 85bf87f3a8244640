"""Key/value shards on the GPU: the summands that sigattn_fwd_shard / sigattn_bwd_shard
give for contiguous shards of one long sequence add up to the oracle's attention against
the whole sequence.  The shards run one after the other on one GPU (no kernel waits for
another); the exchange between ranks is covered by the CPU test with gloo."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_04431_b200 import inputs, sharding
from parity_util import BF16_REL_FRO, rel_fro, to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,H_kv,N,D,world,causal,with_slopes", [
    (1, 4, 4, 1000, 128, 4, True, False),    # ragged shards of 250 keys: masks cut through tiles at odd offsets
    (2, 4, 2, 700, 64, 3, True, True),       # grouped heads, ALiBi distances across shards
    (1, 2, 2, 512, 128, 2, False, False),    # no mask: every shard is a plain summand
])
def test_shard_summands_add_up(B, H, H_kv, N, D, world, causal, with_slopes):
    import torch
    import paper_2409_04431_b200 as sa
    q, _, _, d_o = inputs.random_case(B, H, N, D, 101)
    _, k, v, _ = inputs.random_case(B, H_kv, N, D, 102)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale, bias = 1.0 / math.sqrt(D), -math.log(N)
    o_sum = torch.zeros(tq.shape, dtype=torch.float32, device="cuda")
    dq_sum = torch.zeros_like(o_sum)
    dk = torch.empty_like(tk)
    dv = torch.empty_like(tv)
    for rank in range(world):
        rows = sharding.kv_shard_range(N, world, rank)
        ks, vs = tk[:, :, rows.start:rows.stop].contiguous(), tv[:, :, rows.start:rows.stop].contiguous()
        o_sum += sharding.kv_sharded_fwd(lambda a, b, c, pos0: sa.sigattn_fwd_shard(a, b, c, scale, bias, pos0, causal, sl),
                                         tq, ks, vs, rows.start).float()
        g = sharding.kv_sharded_bwd(lambda a, b, c, d, pos0: sa.sigattn_bwd_shard(a, b, c, d, scale, bias, pos0, causal, sl),
                                    tq, ks, vs, tdo, rows.start)
        dq_sum += g[0].float()
        dk[:, :, rows.start:rows.stop] = g[1]
        dv[:, :, rows.start:rows.stop] = g[2]
    sa.sigattn_check()
    ref_o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes)
    ref_dq, ref_dk, ref_dv = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes)
    # each summand is rounded to bf16 once, so the sum of `world` summands carries a little more
    # rounding noise than one bf16 result
    tol = BF16_REL_FRO * math.sqrt(2.0)
    assert rel_fro(to_host(o_sum), ref_o) < tol
    assert rel_fro(to_host(dq_sum), ref_dq) < tol
    assert rel_fro(to_host(dk), ref_dk) < BF16_REL_FRO
    assert rel_fro(to_host(dv), ref_dv) < BF16_REL_FRO


def test_shard_entirely_after_the_queries_gives_zeros():
    import torch
    import paper_2409_04431_b200 as sa
    q, k, v, d_o = (to_device(t, "bf16") for t in inputs.random_case(1, 2, 300, 64, seed=7))
    o = sa.sigattn_fwd_shard(q, k, v, 0.125, -5.0, -300, causal=True)        # the shard starts 300 positions later
    dq, dk, dv, _ = sa.sigattn_bwd_shard(q, k, v, d_o, 0.125, -5.0, -300, causal=True)
    sa.sigattn_check()
    for t in (o, dq, dk, dv):
        assert torch.count_nonzero(t).item() == 0
    # one position of overlap: only the last query sees only the first key
    o1 = sa.sigattn_fwd_shard(q, k, v, 0.125, -5.0, -299, causal=True)
    assert torch.count_nonzero(o1[:, :, :299]).item() == 0 and torch.count_nonzero(o1[:, :, 299]).item() > 0


@pytest.mark.parametrize("B,H,H_kv,N,D,world,causal,with_slopes", [
    (1, 4, 4, 1000, 128, 4, True, False),
    (2, 4, 2, 700, 64, 3, True, True),
    (1, 2, 2, 40, 64, 2, True, False),       # few queries per owner: the packed small-query path accumulates too
    (1, 2, 2, 512, 128, 2, False, False),
])
def test_shards_add_into_the_owners_accumulators(B, H, H_kv, N, D, world, causal, with_slopes):
    """The fused form: every shard adds its summands of O and dQ, in fp32, into the accumulator of
    the rank that owns the query rows; the owners convert at the end.  One GPU plays all ranks in
    turn (on several GPUs the accumulators would be peer mappings)."""
    import torch
    import paper_2409_04431_b200 as sa
    q, _, _, d_o = inputs.random_case(B, H, N, D, 103)
    _, k, v, _ = inputs.random_case(B, H_kv, N, D, 104)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32) if with_slopes else None
    tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
    sl = None if slopes is None else torch.from_numpy(slopes).cuda()
    scale, bias = 1.0 / math.sqrt(D), -math.log(N)
    owners = [sharding.kv_shard_range(N, world, r) for r in range(world)]       # query rows per owner
    q_sl = [tq[:, :, r.start:r.stop].contiguous() for r in owners]
    do_sl = [tdo[:, :, r.start:r.stop].contiguous() for r in owners]
    starts = [r.start for r in owners]
    o_acc = [torch.zeros(t.shape, dtype=torch.float32, device="cuda") for t in q_sl]
    dq_acc = [torch.zeros(t.shape, dtype=torch.float32, device="cuda") for t in q_sl]
    dk = torch.empty_like(tk)
    dv = torch.empty_like(tv)
    for rank in range(world):
        rows = sharding.kv_shard_range(N, world, rank)
        ks, vs = tk[:, :, rows.start:rows.stop].contiguous(), tv[:, :, rows.start:rows.stop].contiguous()
        sharding.kv_sharded_fwd_acc(
            lambda a, b, c, acc, pos0: sa.sigattn_fwd_shard_acc(a, b, c, acc, scale, bias, pos0, causal, sl),
            q_sl, starts, ks, vs, rows.start, o_acc)
        g = sharding.kv_sharded_bwd_acc(
            lambda a, b, c, d, acc, gk, gv, pos0: sa.sigattn_bwd_shard_acc_kv(a, b, c, d, acc, gk, gv, scale, bias, pos0,
                                                                            causal, sl),
            q_sl, do_sl, starts, ks, vs, rows.start, dq_acc, torch.full_like(ks, float("nan")),
            torch.full_like(vs, float("nan")))
        dk[:, :, rows.start:rows.stop], dv[:, :, rows.start:rows.stop] = g
    o = torch.cat([sa.sigattn_acc_to_bf16(a) for a in o_acc], dim=2)
    dq = torch.cat([sa.sigattn_acc_to_bf16(a, scale) for a in dq_acc], dim=2)
    sa.sigattn_check()
    ref_o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes)
    ref_dq, ref_dk, ref_dv = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes)
    # the sums are formed in fp32 and rounded to bf16 once: the plain tolerance holds
    assert rel_fro(to_host(o), ref_o) < BF16_REL_FRO
    assert rel_fro(to_host(dq), ref_dq) < BF16_REL_FRO
    # dK, dV of a shard: one bf16 summand per owner, added by the kernels (bf16 reduce-adds)
    tol = BF16_REL_FRO * math.sqrt(2.0)
    assert rel_fro(to_host(dk), ref_dk) < tol
    assert rel_fro(to_host(dv), ref_dv) < tol
