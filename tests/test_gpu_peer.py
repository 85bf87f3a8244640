"""Keys and values sharded over two PROCESSES that add their summands of O and dQ straight into
the accumulator of the process that owns the query rows, through CUDA inter-process mappings
(sharding.PeerAccumulators over sigattn_peer_export / sigattn_peer_open): the part of the
multi-GPU path that needs no second GPU to be exercised.  With two or more GPUs each process takes
its own; with one, both share it (no kernel here waits for another, so that is safe)."""
import math
import os
import socket

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

B, H, N, D = 1, 4, 900, 128
SCALE, BIAS = 1.0 / math.sqrt(D), -math.log(N)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import torch
    import torch.distributed as dist
    import oracle  # noqa: F401  (not used here: the parent compares)
    import paper_2409_04431_b200 as sa
    from paper_2409_04431_b200 import inputs, sharding
    from parity_util import to_device

    torch.cuda.set_device(rank % torch.cuda.device_count())
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        q, k, v, d_o = inputs.random_case(B, H, N, D, seed=4100)
        slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32)
        sl = torch.from_numpy(slopes).cuda()
        owners = [sharding.kv_shard_range(N, world, r) for r in range(world)]   # query rows per owner
        mine = owners[rank]
        tq, tk, tv, tdo = (to_device(t, "bf16") for t in (q, k, v, d_o))
        q_sl = [tq[:, :, r.start:r.stop].contiguous() for r in owners]
        do_sl = [tdo[:, :, r.start:r.stop].contiguous() for r in owners]
        ks, vs = tk[:, :, mine.start:mine.stop].contiguous(), tv[:, :, mine.start:mine.stop].contiguous()
        # one allocation per rank: [0] the O accumulator, [1] the dQ accumulator of the rows it owns
        n_own = [r.stop - r.start for r in owners]
        acc = torch.zeros((2, B, H, n_own[rank], D), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        peers = sharding.PeerAccumulators(acc)
        dist.barrier()                                  # every accumulator is cleared and mapped
        half = [B * H * n * D * 4 for n in n_own]       # bytes of one accumulator of each owner
        o_addr = [peers.address(r, 0) for r in range(world)]
        dq_addr = [peers.address(r, half[r]) for r in range(world)]
        sharding.kv_sharded_fwd_acc(
            lambda a, b, c, dst, pos0: sa.sigattn_fwd_shard_acc(a, b, c, dst, SCALE, BIAS, pos0, True, sl),
            q_sl, [r.start for r in owners], ks, vs, mine.start, o_addr)
        dk, dv = sharding.kv_sharded_bwd_acc(
            lambda a, b, c, d, dst, gk, gv, pos0: sa.sigattn_bwd_shard_acc_kv(a, b, c, d, dst, gk, gv, SCALE, BIAS, pos0,
                                                                            True, sl),
            q_sl, do_sl, [r.start for r in owners], ks, vs, mine.start, dq_addr, torch.empty_like(ks),
            torch.empty_like(vs))
        peers.all_added()
        o = sa.sigattn_acc_to_bf16(acc[0])
        dq = sa.sigattn_acc_to_bf16(acc[1], SCALE)
        sa.sigattn_check()
        np.savez(os.path.join(out_dir, f"peer{rank}.npz"), o=o.float().cpu().numpy(), dq=dq.float().cpu().numpy(),
                 dk=dk.float().cpu().numpy(), dv=dv.float().cpu().numpy(), lo=mine.start, hi=mine.stop)
        dist.barrier()                                  # nobody unmaps while another rank still reads
        peers.close()
    finally:
        dist.destroy_process_group()


def test_two_processes_add_into_each_others_accumulators(tmp_path):
    import torch.multiprocessing as mp
    import oracle
    from paper_2409_04431_b200 import inputs
    from parity_util import BF16_REL_FRO, rel_fro
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    q, k, v, d_o = inputs.random_case(B, H, N, D, seed=4100)
    slopes = (0.5 ** np.arange(1, H + 1)).astype(np.float32)
    ref_o = oracle.sigattn_fwd(q, k, v, SCALE, BIAS, True, slopes)
    ref_dq, ref_dk, ref_dv = oracle.sigattn_bwd(q, k, v, d_o, SCALE, BIAS, True, slopes)
    covered = []
    for rank in range(world):
        r = np.load(tmp_path / f"peer{rank}.npz")
        lo, hi = int(r["lo"]), int(r["hi"])
        assert np.all(np.isfinite(r["o"])) and np.all(np.isfinite(r["dq"]))
        assert rel_fro(r["o"], ref_o[:, :, lo:hi]) < BF16_REL_FRO
        assert rel_fro(r["dq"], ref_dq[:, :, lo:hi]) < BF16_REL_FRO
        tol = BF16_REL_FRO * math.sqrt(2.0)             # one bf16 summand per owner of query rows
        assert rel_fro(r["dk"].astype(np.float64), ref_dk[:, :, lo:hi]) < tol
        assert rel_fro(r["dv"].astype(np.float64), ref_dv[:, :, lo:hi]) < tol
        covered += list(range(lo, hi))
    assert covered == list(range(N))
