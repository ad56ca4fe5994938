"""GPU parity of the recursion steered by a budget (Sailor Sec. 4.2.3): sailor_plan_dp with
SAILOR_DP_FLAG_BUDGET_LOOP against the oracle's limited recursion on the same seeded inputs.  Types, zones,
problem indices and counts bit-exact; the recursion's value, t_iter and cost within 1e-5 relative, and identical
in their bits."""
import ctypes as C
import glob
import itertools
import json
import os

import numpy as np
import pytest

from helpers import GOLDEN, REL_TOL_F64, rel_close, workload_from_tables
from oracle.binding import Oracle
from paper_2504_17096_b200 import binding as B
from paper_2504_17096_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _needs_cuda():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")


class Ctx:
    def __init__(self, w):
        self.ctx = B.sailor_create(w, 0, 0)
        B.sailor_set_availability(self.ctx, w.avail)
        self.space = B.make_space(w)

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        B.sailor_destroy(self.ctx)


def configs_of(w):
    return list(itertools.product(w.p_values, w.mbs_idx, w.tp_idx, w.rc_values, w.d_values))


def oracle_limited(w, o, orders, limit):
    """Every problem by the oracle's limited recursion: ([(value, problem index, result, simulated)] of the plans
    whose simulated cost is within the limit, number of problems with a plan, number over the limit)."""
    kept, solved, over = [], 0, 0
    for c, (P, mi, ti, rc, D) in enumerate(configs_of(w)):
        for j, zl in enumerate(orders):
            r = o.solve_dp_budget(P, mi, ti, rc, D, zl, limit)
            if r is None:
                continue
            solved += 1
            sim = o.simulate(r["plan"])
            assert sim.status == 0
            if sim.cost > limit:
                over += 1
                continue
            kept.append((r["value"], c * len(orders) + j, r, sim))
    kept.sort(key=lambda x: (x[0], x[1]))
    return kept, solved, over


def assert_same(res, st, want, solved, over, w, orders, k, what):
    assert st.n_problems == len(configs_of(w)) * len(orders) and st.n_unfinished == 0, what
    assert (st.n_solved, st.n_over_constraint) == (solved, over), what
    assert [(r.config * len(orders) + r.order) for r in res] == [x[1] for x in want[:k]], what
    for r, (value, _, ref, sim) in zip(res, want):
        assert list(r.type[: r.P]) == ref["types"] and list(r.zone[: r.P]) == ref["zones"], what
        assert r.status == 0 and r.peak_mem == sim.peak_mem, what
        assert rel_close([r.value, r.t_iter, r.cost], [value, sim.t_iter, sim.cost], REL_TOL_F64), what
        assert (r.value, r.t_iter, r.cost) == (value, sim.t_iter, sim.cost), what            # identical bits


def test_hand_worked_limited_recursion():
    for path in sorted(glob.glob(os.path.join(GOLDEN, "dp_budget", "*.json"))):
        with open(path) as f:
            case = json.load(f)
        w = workload_from_tables(case["tables"], case["name"])
        p, e = case["problem"], case["expect"]
        w.p_values, w.mbs_idx, w.tp_idx, w.rc_values, w.d_values = [p["P"]], [p["mbs_idx"]], [p["tp_idx"]], [p["rc"]], [p["D"]]
        with Ctx(w) as cx:
            res, st = B.sailor_plan_dp(cx.ctx, cx.space, [p["zone_list"]], 4, budget=p["limit"], budget_loop=True)
            assert st.n_solved == 1 and st.n_unfinished == 0
            if e["simulated_cost"] <= p["limit"]:
                assert len(res) == 1 and st.n_over_constraint == 0
                assert list(res[0].type[: p["P"]]) == e["types"] and list(res[0].zone[: p["P"]]) == e["zones"]
                assert res[0].value == pytest.approx(e["value"], rel=1e-12)
                assert res[0].cost == pytest.approx(e["simulated_cost"], rel=1e-12)
                # without the loop the recursion's plan is the unlimited one, and the check of the budget drops it
                plain, pst = B.sailor_plan_dp(cx.ctx, cx.space, [p["zone_list"]], 4, budget=p["limit"])
                assert plain == [] and pst.n_solved == 1 and pst.n_over_constraint == 1
            else:                       # the plan the loop finds is within its own charge, over the simulator's cost
                assert res == [] and st.n_over_constraint == 1
            for limit in e["no_plan_limits"]:
                none, nst = B.sailor_plan_dp(cx.ctx, cx.space, [p["zone_list"]], 4, budget=limit, budget_loop=True)
                assert none == [] and nst.n_solved == 0


def _tiny():
    yield W.tiny(seed=3, n_types=3, n_zones=2, L=6, p_values=[1, 2, 3, 6]), [[0, 1], [1, 0], [1]]
    yield W.tiny(seed=7, n_types=2, n_zones=3, L=5, p_values=[2, 4, 5], d_values=(1, 2, 4)), [[0, 1, 2], [2, 0], [1]]
    yield W.tiny(seed=8, n_types=4, n_zones=1, L=4, p_values=[1, 3, 4], d_values=(1, 3)), [[0]]
    yield (W.tiny(seed=14, n_types=8, n_zones=2, L=12, p_values=[6, 5], d_values=(4, 8), tp_values=(1, 2), mbs_values=(1, 4)),
           [[1, 0], [0]])


@pytest.mark.parametrize("w,orders", list(_tiny()), ids=lambda x: getattr(x, "name", None))
def test_budget_loop_matches_oracle_on_tiny_clusters(w, orders):
    o = Oracle(w)
    # limits spread over the costs of the plans the unlimited recursion finds: some cut nothing, some nearly all
    costs = []
    for c, (P, mi, ti, rc, D) in enumerate(configs_of(w)):
        r = o.solve_dp(P, mi, ti, rc, D, orders[0])
        if r is not None:
            costs.append(o.simulate(r["plan"]).cost)
    assert len(costs) > 4
    costs.sort()
    with Ctx(w) as cx:
        seen_cut = 0
        for limit in (costs[0] * 0.7, costs[len(costs) // 4], costs[len(costs) // 2] * 1.001, costs[-1] * 3.0):
            want, solved, over = oracle_limited(w, o, orders, limit)
            for k in (1, 32):
                res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, k, budget=limit, budget_loop=True)
                assert_same(res, st, want, solved, over, w, orders, k, f"{w.name} limit={limit} k={k}")
            seen_cut += solved < sum(1 for _ in configs_of(w)) * len(orders)
        assert seen_cut > 0


def test_budget_loop_on_workload_2_up_to_eight_stages():
    """Workload 2's model and cluster (3 types, 2 zones), pipelines of up to 8 stages, every zone order: the limit
    at 1.2 x the cheapest plan the unlimited recursion finds, as the workload's own budget rule has it."""
    w = W.config2()
    w.p_values = [p for p in w.p_values if p <= 8]
    orders = B.all_zone_orders(w.n_zones)
    o = Oracle(w)
    cheapest = min(o.simulate(r["plan"]).cost
                   for P, mi, ti, rc, D in configs_of(w) for zl in orders
                   for r in [o.solve_dp(P, mi, ti, rc, D, zl)] if r is not None)
    limit = 1.2 * cheapest
    want, solved, over = oracle_limited(w, o, orders, limit)
    assert len(want) > 8 and solved > len(want)
    with Ctx(w) as cx:
        res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, 16, budget=limit, budget_loop=True)
        assert_same(res, st, want, solved, over, w, orders, 16, "cfg2 P<=8")
        # the loop keeps problems alive that the plain check of the budget loses
        plain, pst = B.sailor_plan_dp(cx.ctx, cx.space, orders, 16, budget=limit)
        assert st.n_solved - st.n_over_constraint >= pst.n_solved - pst.n_over_constraint


def test_budget_loop_argument_checks():
    w = W.tiny(seed=3)
    with Ctx(w) as cx:
        with pytest.raises(B.SailorError) as e:
            B.sailor_plan_dp(cx.ctx, cx.space, [[0]], 4, budget=0.0, budget_loop=True)
        assert e.value.code == B.E_ARG
    deep = W.tiny(seed=31, n_types=2, n_zones=2, L=96, p_values=[48], d_values=(1,), tp_values=(1,), mbs_values=(1,), gbs=64)
    with Ctx(deep) as cx:
        with pytest.raises(B.SailorError) as e:
            B.sailor_plan_dp(cx.ctx, cx.space, [[0]], 4, budget=1.0, budget_loop=True)
        assert e.value.code == B.E_RANGE
