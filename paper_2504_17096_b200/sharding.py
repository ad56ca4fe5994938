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


def subspace_costs(w) -> List[Tuple[int, float]]:
    """(candidates, relative cost of one candidate) of each pipeline depth's sub-space, in flat-index order.
    A candidate costs its fixed part plus one step per stage of the last segment (the search keeps the running
    sums of the other segments per prefix), which is how the measured per-depth times of the search scale."""
    base = len(w.mbs_idx) * len(w.tp_idx) * len(w.rc_values) * len(w.d_values)
    out = []
    for p in w.p_values:
        nseg = min(p, w.seg_max)
        last = p - ((nseg - 1) * p + nseg - 1) // nseg          # stages of the last segment
        out.append((base * w.radix ** nseg, COST_FIXED + COST_PER_STAGE * last))
    return out


# Fitted to the search times of workload 5's sub-spaces of equal size (pipelines of 4, 6, 8, 12, 16 stages: 1, 1, 2, 3, 4
# stages in the last segment; 2.67, 2.69, 2.87, 3.03, 3.11 ms on one B200): time = 2.53 + 0.15 x stages.
COST_FIXED, COST_PER_STAGE = 17.0, 1.0


def split_by_cost(parts: Sequence[Tuple[int, float]], world: int, rank: int) -> Tuple[int, int]:
    """Contiguous [lo, hi) of rank `rank`: the flat range [0, sum of sizes) cut where the estimated cost
    (size x weight, summed over consecutive parts) reaches rank / world and (rank + 1) / world of the total.
    The ranges of all ranks tile the space exactly."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("bad world/rank")
    total = sum(n * wgt for n, wgt in parts)
    n_all = sum(n for n, _ in parts)

    def cut(j: int) -> int:
        if j <= 0:
            return 0
        if j >= world:
            return n_all
        want, flat, cost = total * j / world, 0, 0.0
        for n, wgt in parts:
            if cost + n * wgt >= want and wgt > 0:
                return min(n_all, flat + int((want - cost) / wgt))
            flat += n
            cost += n * wgt
        return n_all

    return cut(rank), cut(rank + 1)


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
