"""Host-side helpers for splitting one search space over several GPUs.

Candidates are independent, so a space is cut into contiguous flat-index ranges, each rank runs
`sailor_plan_range` on its own GPU, and the per-rank top-k lists are merged by (score, flat).
The only exchange is k small records per rank; there is no data-path collective.

The dynamic-programming search shards by zone order: its problems (configuration x zone order) are
independent, a rank solves every configuration for its slice of the order list with `sailor_plan_dp`,
and the per-rank lists are merged by (value, problem index) with the order index made global."""
from __future__ import annotations

from typing import List, Sequence, Tuple


def split_range(n: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced [lo, hi) of rank `rank` out of `world`; ranges tile [0, n) exactly."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("bad world/rank")
    return n * rank // world, n * (rank + 1) // world


def merge_topk(lists: Sequence[Sequence[Tuple[float, int]]], k: int) -> List[Tuple[float, int]]:
    """Merge per-range lists of (score, flat) pairs; ascending, ties to the lowest flat index."""
    allp = [tuple(p) for l in lists for p in l]
    allp.sort()
    return allp[:k]


def sum_counts(counts: Sequence[dict]) -> dict:
    """Add the class counts of the ranges; the cheapest feasible cost is the minimum over ranges."""
    out: dict = {}
    for c in counts:
        for key, v in c.items():
            if key == "min_feasible_cost":
                continue
            out[key] = out.get(key, 0) + v
    costs = [c["min_feasible_cost"] for c in counts if c.get("n_feasible")]
    out["min_feasible_cost"] = min(costs) if costs else 0.0
    return out


def gather_and_merge(local: Sequence[Tuple[float, int]], local_counts: dict, k: int, group=None):
    """All ranks contribute their list and counts; every rank gets the merged result."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    lists: list = [None] * world
    counts: list = [None] * world
    dist.all_gather_object(lists, list(local), group=group)
    dist.all_gather_object(counts, dict(local_counts), group=group)
    return merge_topk(lists, k), sum_counts(counts)


def split_zone_orders(orders: Sequence[Sequence[int]], world: int, rank: int):
    """The slice of the zone-order list that rank `rank` solves: (index of its first order, its orders)."""
    lo, hi = split_range(len(orders), world, rank)
    return lo, [list(o) for o in orders[lo:hi]]


def merge_dp(lists: Sequence[Sequence[Tuple[float, int, int]]], n_orders_total: int, k: int) -> List[Tuple[float, int, int]]:
    """Merge per-rank lists of (value, configuration, global order index): ascending by value, ties to the
    lowest problem index = configuration * n_orders_total + order, as one call over all orders would rank them."""
    allp = [tuple(p) for l in lists for p in l]
    allp.sort(key=lambda p: (p[0], p[1] * n_orders_total + p[2]))
    return allp[:k]
