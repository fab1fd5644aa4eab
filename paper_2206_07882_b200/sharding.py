"""Utterance sharding across one-process-per-GPU ranks.

Utterances are independent, so the path shards by utterance with replicated weights and no
data-path collective.  The only communication is the reduction of the step time (max over
ranks) used for reporting; it works with any torch.distributed backend (nccl on GPUs, gloo
in the CPU tests)."""
from __future__ import annotations

from typing import Tuple


def shard_range(n_items: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [lo, hi) slice of n_items owned by `rank`; sizes differ by at most one."""
    base, extra = divmod(n_items, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic utterances of one rank under weak scaling (fixed batch per GPU)."""
    return base_seed + 1000 * rank


def job_time_ms(local_ms: float, device=None) -> float:
    """Whole-job time of a step: the slowest rank's device time."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rtf(local_ms: float, utterances_per_rank: int, seconds_per_utterance: float,
                  world: int, device=None) -> float:
    """Real-time factor of the whole job: max-over-ranks time / audio processed by all ranks."""
    return (job_time_ms(local_ms, device) / 1e3) / (world * utterances_per_rank * seconds_per_utterance)
