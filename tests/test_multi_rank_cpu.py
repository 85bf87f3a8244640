"""The N > 1 path of the benchmark on CPU: two gloo ranks check the sharding rules and the
max-over-ranks timing reduction (the attention path itself has no collective)."""
import os
import socket

import numpy as np
import pytest


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    from paper_2409_04431_b200 import inputs, sharding

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = inputs.CONFIGS["c1"]
        # each rank draws its own batch
        q, *_ = inputs.make_inputs(cfg, seed=sharding.rank_seed(cfg, rank))
        # per-rank "device times": rank 1 is the slow one
        local = [10.0 + 5.0 * rank, 3.0 + rank, 7.0 - rank]
        red = sharding.max_over_ranks(local)
        np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array(red + [float(q[0, 0, 0, 0])]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timings_to_the_slowest_rank(tmp_path):
    import torch.multiprocessing as mp
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = np.load(tmp_path / "r0.npy"), np.load(tmp_path / "r1.npy")
    np.testing.assert_array_equal(r0[:3], [15.0, 4.0, 7.0])   # element-wise max over both ranks
    np.testing.assert_array_equal(r1[:3], r0[:3])
    assert r0[3] != r1[3]                                      # different seeds -> different batches


def test_sharding_rules():
    from paper_2409_04431_b200 import inputs, sharding
    # strong-scaling split of (batch, head) pairs: contiguous, disjoint, complete, balanced
    for total, world in [(32, 8), (32, 3), (5, 8), (384, 7)]:
        seen = []
        sizes = []
        for r in range(world):
            rg = sharding.shard_heads(total, world, r)
            seen += list(rg)
            sizes.append(len(rg))
        assert seen == list(range(total))
        assert max(sizes) - min(sizes) <= 1
    cfg = inputs.CONFIGS["c4"]
    assert sharding.rank_seed(cfg, 0) == inputs.SEED_BASE + 4
    assert len({sharding.rank_seed(cfg, r) for r in range(8)}) == 8
    # weak scaling: N ranks, same per-rank work, same time -> N times the throughput
    one = sharding.whole_job_tflops(1e12, 10, 1, 100.0)
    assert sharding.whole_job_tflops(1e12, 10, 8, 100.0) == pytest.approx(8 * one)
    assert one == pytest.approx(100.0)
    # without a process group the reduction is the identity
    assert sharding.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]


def _kv_worker(rank, world, port, out_dir):
    """Each rank holds one contiguous key/value shard of the same sequence; the per-shard
    computation is the float64 oracle standing in for the CUDA entry points."""
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2409_04431_b200 import sharding

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, H, N, D = 1, 2, 11, 4
        rng = np.random.default_rng(5)                      # the same sequence on every rank
        q, k, v, d_o = (rng.standard_normal((B, H, N, D)) for _ in range(4))
        slopes = np.array([0.5, 0.25])
        scale, bias = 0.5, -1.0
        rows = sharding.kv_shard_range(N, world, rank)
        ks, vs = k[:, :, rows.start:rows.stop], v[:, :, rows.start:rows.stop]

        def attend(a, b, c, pos0):
            return torch.from_numpy(oracle.sigattn_fwd(a.numpy(), b.numpy(), c.numpy(), scale, bias, True, slopes, pos0=pos0))

        def attend_bwd(a, b, c, d, pos0):
            return tuple(torch.from_numpy(g) for g in
                         oracle.sigattn_bwd(a.numpy(), b.numpy(), c.numpy(), d.numpy(), scale, bias, True, slopes, pos0=pos0))

        tq, tks, tvs, tdo = (torch.from_numpy(np.ascontiguousarray(t)) for t in (q, ks, vs, d_o))
        o = sharding.kv_sharded_fwd(attend, tq, tks, tvs, rows.start)
        dq, dk, dv = sharding.kv_sharded_bwd(attend_bwd, tq, tks, tvs, tdo, rows.start)
        np.savez(os.path.join(out_dir, f"kv{rank}.npz"), o=o.numpy(), dq=dq.numpy(), dk=dk.numpy(), dv=dv.numpy(),
                 lo=rows.start, hi=rows.stop)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_sum_key_value_shards(tmp_path):
    """O and dQ after the all-reduce equal the attention against the whole sequence on every
    rank; dK, dV of each rank are the slices of the whole gradient."""
    import torch.multiprocessing as mp
    import oracle
    world, port = 2, _free_port()
    mp.spawn(_kv_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    rng = np.random.default_rng(5)
    q, k, v, d_o = (rng.standard_normal((1, 2, 11, 4)) for _ in range(4))
    slopes = np.array([0.5, 0.25])
    ref_o = oracle.sigattn_fwd(q, k, v, 0.5, -1.0, True, slopes)
    ref_dq, ref_dk, ref_dv = oracle.sigattn_bwd(q, k, v, d_o, 0.5, -1.0, True, slopes)
    covered = []
    for rank in range(world):
        r = np.load(tmp_path / f"kv{rank}.npz")
        # the exchange adds in float32
        np.testing.assert_allclose(r["o"], ref_o, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(r["dq"], ref_dq, rtol=1e-5, atol=1e-6)
        lo, hi = int(r["lo"]), int(r["hi"])
        np.testing.assert_allclose(r["dk"], ref_dk[:, :, lo:hi], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(r["dv"], ref_dv[:, :, lo:hi], rtol=1e-12, atol=1e-14)
        covered += list(range(lo, hi))
    assert covered == list(range(11))


def test_fused_shard_sum_host_logic_with_shared_accumulators():
    """kv_sharded_fwd_acc / kv_sharded_bwd_acc: every rank adds, for every owner of query rows,
    into that owner's accumulator with the right position offset.  Three ranks are played in turn
    in one process (the accumulators stand for peer-mapped memory), the oracle is the local call."""
    import torch
    import oracle
    from paper_2409_04431_b200 import sharding
    world, B, H, N, D = 3, 1, 2, 13, 4
    rng = np.random.default_rng(9)
    q, k, v, d_o = (rng.standard_normal((B, H, N, D)) for _ in range(4))
    slopes = np.array([0.5, 0.25])
    scale, bias = 0.5, -1.0

    def attend_acc(a, b, c, acc, pos0):
        acc += torch.from_numpy(oracle.sigattn_fwd(a.numpy(), b.numpy(), c.numpy(), scale, bias, True, slopes, pos0=pos0))

    def attend_bwd_acc(a, b, c, d, acc, dk_sum, dv_sum, pos0):
        dq, dk, dv = oracle.sigattn_bwd(a.numpy(), b.numpy(), c.numpy(), d.numpy(), scale, bias, True, slopes, pos0=pos0)
        acc += torch.from_numpy(dq)
        dk_sum += torch.from_numpy(dk)
        dv_sum += torch.from_numpy(dv)

    owners = [sharding.kv_shard_range(N, world, r) for r in range(world)]
    cut = lambda t, r: torch.from_numpy(np.ascontiguousarray(t[:, :, r.start:r.stop]))
    q_sl, do_sl = [cut(q, r) for r in owners], [cut(d_o, r) for r in owners]
    starts = [r.start for r in owners]
    o_acc = [torch.zeros_like(t) for t in q_sl]
    dq_acc = [torch.zeros_like(t) for t in q_sl]
    dk, dv = np.zeros_like(k), np.zeros_like(v)
    for rank in range(world):
        rows = sharding.kv_shard_range(N, world, rank)
        sharding.kv_sharded_fwd_acc(attend_acc, q_sl, starts, cut(k, rows), cut(v, rows), rows.start, o_acc)
        ks, vs = cut(k, rows), cut(v, rows)
        g = sharding.kv_sharded_bwd_acc(attend_bwd_acc, q_sl, do_sl, starts, ks, vs, rows.start, dq_acc,
                                        torch.full_like(ks, 7.0), torch.full_like(vs, 7.0))   # (cleared by the helper)
        dk[:, :, rows.start:rows.stop], dv[:, :, rows.start:rows.stop] = g[0].numpy(), g[1].numpy()
    ref_o = oracle.sigattn_fwd(q, k, v, scale, bias, True, slopes)
    ref = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, True, slopes)
    np.testing.assert_allclose(torch.cat(o_acc, dim=2).numpy(), ref_o, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(torch.cat(dq_acc, dim=2).numpy(), ref[0], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(dk, ref[1], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(dv, ref[2], rtol=1e-12, atol=1e-14)
