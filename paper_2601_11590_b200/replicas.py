"""Data-parallel replicas of the encoder: which GPU encodes which item.

Items (images, clips) are independent units of the Encode stage: attention is block-diagonal and every
other step is row-wise, so a batch can be split across replicas with no collective on the data path;
each replica writes the feature rows of its own items.  The split should balance cost, not item
count: an item of n tokens costs about a*n (linear layers) + b*n^2 (attention).  The assignment below
is the least-loaded-first rule the paper applies to instances (Section 3.4, instance-level dynamic load
balancing) applied to items sorted by decreasing cost (longest processing time first).

Host-side logic only; it has no CUDA dependency.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def item_cost(grid: Sequence[int], hidden: int, mlp: int, layers: int = 1) -> float:
    """Approximate FLOPs of one item: per token 2*(4 h^2 + 2 h m) for the linear layers, 4 h n per token
    for attention over the item's n tokens."""
    t, h, w = (int(v) for v in grid)
    n = t * h * w
    return layers * (2.0 * n * (4.0 * hidden * hidden + 2.0 * hidden * mlp) + 4.0 * hidden * float(n) * n)


def assign_items(grid_thw: Sequence[Sequence[int]], world: int, hidden: int, mlp: int) -> List[List[int]]:
    """Item indices per rank: items in order of decreasing cost, each to the currently least-loaded rank
    (ties to the lowest rank).  Every rank's list is sorted, so a rank encodes its items in batch order."""
    if world < 1:
        raise ValueError("world must be >= 1")
    costs = [item_cost(g, hidden, mlp) for g in grid_thw]
    order = sorted(range(len(costs)), key=lambda i: (-costs[i], i))
    load = [0.0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        out[r].append(i)
        load[r] += costs[i]
    return [sorted(v) for v in out]


def rank_loads(grid_thw: Sequence[Sequence[int]], assignment: Sequence[Sequence[int]], hidden: int, mlp: int
               ) -> List[float]:
    return [sum(item_cost(grid_thw[i], hidden, mlp) for i in items) for items in assignment]


def feature_row_ranges(grid_thw: Sequence[Sequence[int]]) -> List[Tuple[int, int]]:
    """Rows [begin, end) of every item in the whole batch's feature buffer (2x2 merge)."""
    out, row = [], 0
    for t, h, w in grid_thw:
        n = int(t) * (int(h) // 2) * (int(w) // 2)
        out.append((row, row + n))
        row += n
    return out
