"""Multi-rank plumbing of the benchmark: rows (tokens) are independent in every step of the path, so N ranks
run N independent row shards with a replicated layer and there is NO collective on the data path.  The only
communication is the barrier around the timed region and the max-over-ranks of the elapsed time."""
from __future__ import annotations

import os


def env_ranks():
    """(world, rank, local_rank) as torchrun exports them; (1, 0, 0) when launched directly."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def shard_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own rows: same shapes and distributions, different seeds."""
    return base_seed + rank


def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's time: what a whole-job throughput must be divided by."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_step: float, steps: int, elapsed_ms_max: float, world: int) -> float:
    """Weak scaling: every rank processes `units_per_rank_step` per step; the job's rate is the sum over ranks
    divided by the slowest rank's time."""
    return world * units_per_rank_step * steps / (elapsed_ms_max * 1e-3)
