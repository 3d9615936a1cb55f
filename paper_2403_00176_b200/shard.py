"""Multi-GPU: the path shards by independent requests (weights replicated, no collective on the
data path).  One process per GPU; each rank takes a disjoint subset of the seeded batches."""
from __future__ import annotations

from typing import List, Sequence


def assign_batches(n_batches: int, rank: int, world: int) -> List[int]:
    """Round-robin split of batch ids; every rank gets at least one batch."""
    mine = [j for j in range(n_batches) if j % world == rank]
    return mine or [rank % n_batches]


def assign_requests(costs: Sequence[int], world: int) -> List[List[int]]:
    """Greedy longest-first assignment of requests (cost = tokens or pixels) to ranks.
    Returns one list of request indices per rank; the lists partition range(len(costs))."""
    order = sorted(range(len(costs)), key=lambda i: (-costs[i], i))
    load = [0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        out[r].append(i)
        load[r] += costs[i]
    for lst in out:
        lst.sort()
    return out
