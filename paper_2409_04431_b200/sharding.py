"""Multi-GPU plumbing of the benchmark: which rank works on what, and how per-rank timings
become one whole-job number.

The attention path has no exchange step: (batch, head) pairs are independent, so N GPUs run N
independent shards (each rank its own batch, drawn from its own seed) and the only
communication is the timing reduction below.  Kept free of CUDA so that it can be tested with
the gloo backend on CPU.

The second half shards ONE long sequence's keys and values over the ranks (long context):
sigmoid attention has no row normalisation (Section 4), so the attention of all queries
against one contiguous key/value shard is a plain summand of O, and of dQ; ranks exchange one
sum (all-reduce) and no log-sum-exp.  The per-shard computation is the library's
sigattn_fwd_shard / sigattn_bwd_shard; it is passed in, so the exchange logic can be run on
CPU with any stand-in.
"""
from __future__ import annotations

from . import inputs


def rank_seed(cfg: inputs.Config, rank: int) -> int:
    """Seed of the synthetic batch that `rank` generates (rank 0 = the single-GPU batch)."""
    return inputs.SEED_BASE + cfg.index + 1000 * rank


def shard_heads(total_pairs: int, world: int, rank: int) -> range:
    """Contiguous block of (batch, head) pairs owned by `rank` when one fixed problem is
    split over `world` ranks (strong scaling); the first `total_pairs % world` ranks hold
    one pair more."""
    base, extra = divmod(total_pairs, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process
    group): device times are reported as the slowest rank's."""
    import torch
    import torch.distributed as dist

    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_tflops(flops_per_rank_step: float, steps: int, world: int, total_ms_max: float) -> float:
    """Weak scaling: every rank does `flops_per_rank_step` per step; the job's throughput is
    all ranks' work over the slowest rank's device time."""
    return world * flops_per_rank_step * steps / (total_ms_max * 1e-3) / 1e12


def kv_shard_range(n_keys: int, world: int, rank: int) -> range:
    """Contiguous block of key/value rows held by `rank`; the first `n_keys % world` ranks
    hold one row more."""
    return shard_heads(n_keys, world, rank)


def kv_sharded_fwd(attend, q, k_shard, v_shard, key_start: int, query_start: int = 0, group=None):
    """O of all queries `q` against the whole key/value sequence, of which this rank holds
    rows [key_start, key_start + k_shard.shape[2]).

    attend(q, k_shard, v_shard, pos0) -> this rank's summand of O, where pos0 is the position
    of query row 0 relative to the shard's first key (binding.sigattn_fwd_shard with the
    remaining arguments bound).  `query_start`: position of query row 0 in the sequence.
    The summands are added in float32 with one all-reduce over `group`; the result has
    q's dtype.  Without a process group the local summand is returned (one rank)."""
    import torch
    import torch.distributed as dist

    part = attend(q, k_shard, v_shard, query_start - key_start)
    if not (dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1):
        return part
    acc = part.to(torch.float32)
    dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
    return acc.to(part.dtype)


def kv_sharded_bwd(attend_bwd, q, k_shard, v_shard, d_o, key_start: int, query_start: int = 0, group=None):
    """(dQ, dK_shard, dV_shard): dQ is summed over the ranks like O; dK and dV of a shard
    need only that shard's keys and values and stay local.

    attend_bwd(q, k_shard, v_shard, d_o, pos0) -> (dq summand, dk_shard, dv_shard)."""
    import torch
    import torch.distributed as dist

    dq, dk, dv = attend_bwd(q, k_shard, v_shard, d_o, query_start - key_start)[:3]
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        acc = dq.to(torch.float32)
        dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
        dq = acc.to(dq.dtype)
    return dq, dk, dv


def kv_sharded_fwd_acc(attend_acc, q_slices, query_starts, k_shard, v_shard, key_start: int, accumulators):
    """The sum over shards fused into the kernels: this rank adds its shard's summand of O for the
    query rows of every owner straight into that owner's float32 accumulator (on several GPUs a
    peer mapping of it), so no all-reduce follows.

    q_slices[r], query_starts[r]: the query rows rank r owns and the position of their first row;
    accumulators[r]: rank r's accumulator for those rows (tensor or device address), zero before
    the first shard adds.  attend_acc(q, k_shard, v_shard, acc, pos0) is
    binding.sigattn_fwd_shard_acc with the remaining arguments bound.  Every owner converts its
    accumulator (binding.sigattn_acc_to_bf16) once all ranks have added."""
    for q_r, start, acc in zip(q_slices, query_starts, accumulators):
        attend_acc(q_r, k_shard, v_shard, acc, start - key_start)


def kv_sharded_bwd_acc(attend_bwd_acc_kv, q_slices, d_o_slices, query_starts, k_shard, v_shard, key_start: int,
                       accumulators, dk, dv):
    """Backward counterpart: dQ summands go into the owners' accumulators; dK and dV of this rank's
    shard are sums over the owners' query rows and stay local.  Those sums form inside the library
    too: `dk`, `dv` (shaped like the shard) are cleared here and every call adds its summand into them.

    attend_bwd_acc_kv(q, k_shard, v_shard, d_o, dq_acc, dk, dv, pos0) is
    binding.sigattn_bwd_shard_acc_kv with the remaining arguments bound."""
    dk.zero_()
    dv.zero_()
    for q_r, do_r, start, acc in zip(q_slices, d_o_slices, query_starts, accumulators):
        attend_bwd_acc_kv(q_r, k_shard, v_shard, do_r, acc, dk, dv, start - key_start)
    return dk, dv


class PeerAccumulators:
    """The fp32 accumulators of all ranks of `group` as this rank can address them: its own tensor,
    and a peer mapping (an integer device address) of every other rank's.

    Every rank passes the float32 CUDA tensor it owns (zeroed by the caller; any shape, e.g. the O and dQ
    accumulators of its query rows stacked in one allocation - CUDA can map an allocation only once per
    process, so give each rank ONE tensor).  The constructor is collective over `group` (any backend that
    can gather Python objects; the handles are 64 bytes): it exports the local tensor
    (binding.sigattn_peer_export), gathers all exports and opens the others (binding.sigattn_peer_open) on
    this rank's current device.  `address(r, byte_offset)` is what the accumulating shard calls take
    for owner r; `all_added()` orders the conversion after every rank's additions; `close()` unmaps.
    One process per GPU; on one GPU two processes may share it (the kernels never wait on each other)."""

    def __init__(self, local, group=None):
        import torch
        import torch.distributed as dist
        from . import binding

        if not (isinstance(local, torch.Tensor) and local.is_cuda and local.dtype == torch.float32
                and local.is_contiguous()):
            raise ValueError("the local accumulator must be a contiguous float32 CUDA tensor")
        self.group, self.local = group, local
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self._binding = binding
        self._opened = {}
        if self.world == 1:
            return
        handle, offset = binding.sigattn_peer_export(local)
        exports = [None] * self.world
        dist.all_gather_object(exports, (handle, offset), group=group)
        for r, (h, off) in enumerate(exports):
            if r != self.rank:
                self._opened[r] = (binding.sigattn_peer_open(h, off, local.device), off)

    def address(self, owner: int, byte_offset: int = 0) -> int:
        """Device address, valid on this rank, of byte `byte_offset` of owner's accumulator tensor."""
        if owner == self.rank:
            return self.local.data_ptr() + byte_offset
        return self._opened[owner][0] + byte_offset

    def all_added(self, stream=None):
        """Every rank calls this after enqueuing its additions: when it returns on a rank, the adding
        kernels of ALL ranks have finished, and the rank may convert its own accumulator."""
        import torch
        import torch.distributed as dist
        (torch.cuda.current_stream(self.local.device) if stream is None else stream).synchronize()
        if self.world > 1:
            dist.barrier(group=self.group)

    def close(self):
        for address, off in self._opened.values():
            self._binding.sigattn_peer_close(address, off)
        self._opened = {}
