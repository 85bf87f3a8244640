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
