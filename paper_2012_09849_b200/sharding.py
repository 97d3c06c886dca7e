"""Environment partition for multi-GPU runs: contiguous global env-id ranges, no data exchange.

Rows of the actor batch and columns of the rollout storage are independent, so N GPUs run N
replicas of the path on disjoint ranges of global environment ids; an environment's action
depends on (seed, env_id, t) only, hence not on the partition."""
from __future__ import annotations


def env_range(rank: int, world: int, total_envs: int) -> tuple[int, int]:
    """[lo, hi) of the global env ids owned by `rank` when `total_envs` are split over `world` ranks."""
    if not (0 <= rank < world) or total_envs < 0:
        raise ValueError("bad partition")
    base, rem = divmod(total_envs, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def reduce_step_time_ms(local_ms: float, dist=None, device=None) -> float:
    """Max over ranks of a locally measured time (the whole job is as slow as its slowest rank)."""
    if dist is None or not dist.is_initialized():
        return float(local_ms)
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
