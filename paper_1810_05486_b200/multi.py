"""Host-side helpers for running on several GPUs, one process per GPU.

The update of one tensor never needs another tensor, and a tensor's max scans stay local
as long as the tensor is not split.  So a parameter list is spread over ranks by whole
tensors and the data path needs no collective; torch.distributed is only used for the
barrier around a timed region and for the max-over-ranks of its duration.
"""
from typing import List, Sequence


def rank_seed(seed: int, rank: int) -> int:
    """Seed of the synthetic inputs of one rank (weak scaling: every rank its own list)."""
    return seed + 1000 * rank


def partition_tensors(numels: Sequence[int], world: int) -> List[List[int]]:
    """Spread tensor indices over `world` ranks, whole tensors only, balancing element
    counts (largest first onto the lightest rank).  Every index appears exactly once; the
    order inside a rank follows the original list."""
    loads = [0] * world
    parts: List[List[int]] = [[] for _ in range(world)]
    for i in sorted(range(len(numels)), key=lambda j: (-numels[j], j)):
        r = min(range(world), key=lambda k: (loads[k], k))
        parts[r].append(i)
        loads[r] += numels[i]
    return [sorted(p) for p in parts]


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Largest `value` over all ranks (the duration of a timed region is the slowest rank's)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: int, world: int, seconds: float) -> float:
    """Units processed by all ranks together per second of the slowest rank."""
    return units_per_rank * world / seconds
