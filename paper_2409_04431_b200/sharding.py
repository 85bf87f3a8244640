"""Multi-GPU plumbing of the benchmark: which rank works on what, and how per-rank timings
become one whole-job number.

The attention path has no exchange step: (batch, head) pairs are independent, so N GPUs run N
independent shards (each rank its own batch, drawn from its own seed) and the only
communication is the timing reduction below.  Kept free of CUDA so that it can be tested with
the gloo backend on CPU.
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
