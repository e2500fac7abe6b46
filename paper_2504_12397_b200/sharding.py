"""Multi-GPU plumbing of the layer path.  Requests are independent (own tokens, own block-table row, own pages), so
the path shards BY REQUEST with the weights replicated and no collective on the data path; torch.distributed is
used only to agree on a timing (barrier + max over ranks).  Nothing here computes the method's arithmetic."""
from __future__ import annotations

from typing import List, Sequence, Tuple


def partition_requests(n_requests: int, world: int) -> List[Tuple[int, int]]:
    """Contiguous, disjoint [begin, end) request ranges, one per rank, sizes differing by at most one."""
    if world <= 0 or n_requests < 0:
        raise ValueError("world must be positive and n_requests non-negative")
    base, extra = divmod(n_requests, world)
    out, lo = [], 0
    for r in range(world):
        hi = lo + base + (1 if r < extra else 0)
        out.append((lo, hi))
        lo = hi
    return out


def partition_by_tokens(new_tokens: Sequence[int], world: int) -> List[List[int]]:
    """Request indices per rank, balancing the number of new tokens (longest-first greedy); deterministic."""
    loads = [0] * world
    owners: List[List[int]] = [[] for _ in range(world)]
    for i in sorted(range(len(new_tokens)), key=lambda j: (-int(new_tokens[j]), j)):
        r = min(range(world), key=lambda k: (loads[k], k))
        owners[r].append(i)
        loads[r] += int(new_tokens[i])
    return [sorted(o) for o in owners]


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic batch of one rank under weak scaling (every rank draws its own batch)."""
    return int(base_seed) + 7919 * int(rank)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar over the default process group (the value itself when there is no group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds_max: float, world: int) -> float:
    """Whole-job throughput under weak scaling: every rank processed units_per_rank in (at most) seconds_max."""
    return world * units_per_rank / seconds_max
