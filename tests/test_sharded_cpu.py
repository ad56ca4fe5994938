"""The multi-rank host logic (range split, gather, merge) at world size 2 over gloo on CPU.
Each rank evaluates its range with the CPU oracle standing in for its GPU."""
import os
import socket

import pytest
import torch.multiprocessing as mp

from paper_2504_17096_b200 import sharding


def test_split_range_tiles_exactly():
    for n in (0, 1, 7, 6768, 6397205760):
        for world in (1, 2, 3, 8):
            edges = [sharding.split_range(n, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(edges[:-1], edges[1:]))
            sizes = [b - a for a, b in edges]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.split_range(10, 2, 2)


def test_split_by_cost_tiles_exactly_and_balances_the_estimate():
    from paper_2504_17096_b200 import workloads as W
    for w in (W.config5(), W.config3(), W.config1()):
        parts = sharding.subspace_costs(w)
        assert sum(n for n, _ in parts) == w.space_size()
        total = sum(n * c for n, c in parts)
        for world in (1, 2, 3, 8):
            edges = [sharding.split_by_cost(parts, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == w.space_size()
            assert all(a[1] == b[0] for a, b in zip(edges[:-1], edges[1:]))

            def cost(lo, hi):          # estimated cost of [lo, hi)
                out, at = 0.0, 0
                for n, c in parts:
                    out += max(0, min(hi, at + n) - max(lo, at)) * c
                    at += n
                return out
            for lo, hi in edges:
                assert abs(cost(lo, hi) - total / world) <= max(c for _, c in parts) * 2
    with pytest.raises(ValueError):
        sharding.split_by_cost([(10, 1.0)], 2, 2)


def test_merge_topk_breaks_ties_by_flat_index():
    a = [(1.0, 9), (2.0, 3)]
    b = [(1.0, 4), (3.0, 1)]
    assert sharding.merge_topk([a, b], 3) == [(1.0, 4), (1.0, 9), (2.0, 3)]
    assert sharding.merge_topk([[], []], 3) == []


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, q):
    import torch.distributed as dist
    from oracle.binding import Oracle
    from paper_2504_17096_b200 import workloads as W
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.config1()
        o = Oracle(w)
        n = o.space_size()
        lo, hi = sharding.split_range(n, world, rank)
        hits, counts = o.search(w.objective, 8, lo=lo, hi=hi)
        local = [(h["score"], h["flat"]) for h in hits]
        counts = dict(counts)
        counts["min_feasible_cost"] = counts.pop("min_cost")
        merged, total = sharding.gather_and_merge(local, counts, 8)
        q.put((rank, merged, total))
    finally:
        dist.destroy_process_group()


def test_two_ranks_merge_to_the_full_search():
    from oracle.binding import Oracle
    from paper_2504_17096_b200 import workloads as W
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = W.config1()
    full, counts = Oracle(w).search(w.objective, 8)
    want = [(h["score"], h["flat"]) for h in full]
    for rank, merged, total in got:
        assert merged == want
        assert total["n_total"] == counts["n_total"] and total["n_feasible"] == counts["n_feasible"]
        assert total["min_feasible_cost"] == counts["min_cost"]


def _dp_worker(rank, world, port, q):
    import itertools
    import torch.distributed as dist
    from oracle.binding import Oracle
    from paper_2504_17096_b200 import binding as B
    from paper_2504_17096_b200 import workloads as W
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.tiny(seed=7, n_types=2, n_zones=3, L=5, p_values=[2, 4, 5], d_values=(1, 2, 4))
        orders = B.all_zone_orders(w.n_zones)
        lo, mine = sharding.split_zone_orders(orders, world, rank)
        o = Oracle(w)
        local = []
        cfgs = list(itertools.product(w.p_values, w.mbs_idx, w.tp_idx, w.rc_values, w.d_values))
        for c, (P, mi, ti, rc, D) in enumerate(cfgs):          # the oracle stands in for this rank's GPU
            for j, zl in enumerate(mine):
                r = o.solve_dp(P, mi, ti, rc, D, zl)
                if r is not None:
                    local.append((r["value"], c, lo + j))
        local.sort(key=lambda p: (p[0], p[1] * len(orders) + p[2]))
        lists = [None] * world
        dist.all_gather_object(lists, local[:8])
        q.put((rank, sharding.merge_dp(lists, len(orders), 8)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_the_zone_orders_of_the_dp_search():
    import itertools
    from oracle.binding import Oracle
    from paper_2504_17096_b200 import binding as B
    from paper_2504_17096_b200 import workloads as W
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_dp_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = W.tiny(seed=7, n_types=2, n_zones=3, L=5, p_values=[2, 4, 5], d_values=(1, 2, 4))
    orders = B.all_zone_orders(w.n_zones)
    o = Oracle(w)
    full = []
    for c, (P, mi, ti, rc, D) in enumerate(itertools.product(w.p_values, w.mbs_idx, w.tp_idx, w.rc_values, w.d_values)):
        for j, zl in enumerate(orders):
            r = o.solve_dp(P, mi, ti, rc, D, zl)
            if r is not None:
                full.append((r["value"], c, j))
    full.sort(key=lambda p: (p[0], p[1] * len(orders) + p[2]))
    assert len(full) > 8
    for rank, merged in got:
        assert merged == full[:8]
    lo0, a = sharding.split_zone_orders(orders, 2, 0)
    lo1, b = sharding.split_zone_orders(orders, 2, 1)
    assert lo0 == 0 and lo1 == len(a) and a + b == orders
