"""GPU parity of the dynamic-programming search (Sailor Sec. 4.2.2, Eq. 1): sailor_plan_dp against the
oracle's recursion on the same seeded inputs.  Types, zones, problem indices and counts bit-exact; the
recursion's value, t_iter and cost within 1e-5 relative, and identical in their bits."""
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


@pytest.fixture(params=["auto", "dense", "compact", "auto-types", "compact-types", "auto-entries", "compact-entries"], autouse=True)
def _index_mode(request, monkeypatch):
    """Every test runs with each way of indexing the tables' count vectors (mixed radix, by rank, the smaller) and
    with each way of enumerating a stage's work (a thread per reachable count vector for all its types, which is the
    default up to four GPU types; a thread per reachable count vector and type; a thread per table entry)."""
    index, _, enum = request.param.partition("-")
    flags = {"auto": 0, "dense": B.DP_FLAG_INDEX_DENSE, "compact": B.DP_FLAG_INDEX_COMPACT}[index]
    flags |= {"": 0, "types": B.DP_FLAG_ENUM_BY_TYPE, "entries": B.DP_FLAG_ENUM_BY_ENTRY}[enum]
    monkeypatch.setattr(B, "dp_default_flags", flags)
    return index


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
    """Configurations in the order of the library's configuration index."""
    return list(itertools.product(w.p_values, w.mbs_idx, w.tp_idx, w.rc_values, w.d_values))


def oracle_all(w, o, orders):
    """Every problem solved by the oracle: [(value, problem index, result dict)] for those with a plan."""
    out = []
    for c, (P, mi, ti, rc, D) in enumerate(configs_of(w)):
        for j, zl in enumerate(orders):
            r = o.solve_dp(P, mi, ti, rc, D, zl)
            if r is not None:
                out.append((r["value"], c * len(orders) + j, r))
    out.sort(key=lambda x: (x[0], x[1]))
    return out


def assert_dp_equal(res, st, want, w, o, orders, k, what):
    assert st.n_problems == len(configs_of(w)) * len(orders), what
    assert st.n_solved == len(want), what
    assert [(r.config * len(orders) + r.order) for r in res] == [x[1] for x in want[:k]], what
    cfgs = configs_of(w)
    for r, (value, _, ref) in zip(res, want):
        P, mi, ti, rc, D = cfgs[r.config]
        assert (r.P, r.mbs_idx, r.tp_idx, r.rc, r.D) == (P, mi, ti, rc, D), what
        assert list(r.type[:P]) == ref["types"] and list(r.zone[:P]) == ref["zones"], what
        sim = o.simulate(ref["plan"])
        assert r.status == 0 == sim.status and r.peak_mem == sim.peak_mem, what
        assert rel_close([r.value, r.t_iter, r.cost], [value, sim.t_iter, sim.cost], REL_TOL_F64), what
        assert (r.value, r.t_iter, r.cost) == (value, sim.t_iter, sim.cost), what        # identical bits


def test_hand_worked_recursion():
    for path in sorted(glob.glob(os.path.join(GOLDEN, "dp", "*.json"))):
        with open(path) as f:
            case = json.load(f)
        w = workload_from_tables(case["tables"], case["name"])
        p, e = case["problem"], case["expect"]
        w.p_values, w.mbs_idx, w.tp_idx, w.rc_values, w.d_values = [p["P"]], [p["mbs_idx"]], [p["tp_idx"]], [p["rc"]], [p["D"]]
        with Ctx(w) as cx:
            res, st = B.sailor_plan_dp(cx.ctx, cx.space, [p["zone_list"]], 4)
        assert len(res) == 1 and st.n_solved == 1
        assert list(res[0].type[: p["P"]]) == e["types"] and list(res[0].zone[: p["P"]]) == e["zones"]
        assert res[0].value == pytest.approx(e["value"], rel=1e-12)
        assert res[0].t_iter == pytest.approx(e["value"], rel=1e-12)
        if "cost" in e:
            assert res[0].cost == pytest.approx(e["cost"], rel=1e-12)
        for zl in e.get("no_plan_zone_lists", []):
            with Ctx(w) as cx:
                none, st = B.sailor_plan_dp(cx.ctx, cx.space, [zl], 4)
            assert none == [] and st.n_solved == 0


def _tiny():
    yield W.tiny(seed=3, n_types=3, n_zones=2, L=6, p_values=[1, 2, 3, 6]), [[0, 1], [1, 0], [1]]
    yield W.tiny(seed=7, n_types=2, n_zones=3, L=5, p_values=[2, 4, 5], d_values=(1, 2, 4)), [[0, 1, 2], [2, 0], [1]]
    yield W.tiny(seed=8, n_types=4, n_zones=1, L=4, p_values=[1, 3, 4], d_values=(1, 3)), [[0]]
    # the table limits: 8 types (scarce, so the dense tables stay small) and 8 zones
    yield (W.tiny(seed=14, n_types=8, n_zones=2, L=12, p_values=[12, 5], d_values=(4, 8), tp_values=(1, 2), mbs_values=(1, 4)),
           [[1, 0], [0]])
    yield (W.tiny(seed=16, n_types=6, n_zones=8, L=12, p_values=[12, 5], d_values=(2, 4), tp_values=(1, 2), mbs_values=(1, 4)),
           [[7, 6, 5, 4, 3, 2, 1, 0], [2, 5]])
    w = W.tiny(seed=15, n_types=3, n_zones=2, L=40, p_values=[40, 24], d_values=(1, 2), tp_values=(1, 2), mbs_values=(1, 2), gbs=64)
    w.capacity[...] = w.capacity * 6
    yield w, [[0, 1], [1, 0]]


def test_dp_deepest_pipelines_and_bandwidth_polynomials():
    """96 stages (the limit), pipelines that do not divide the layer count, and message-size-dependent links."""
    w = W.tiny(seed=31, n_types=2, n_zones=2, L=96, p_values=[96, 64, 7], d_values=(1, 2), tp_values=(1, 2),
               mbs_values=(1, 2), gbs=64)
    w.capacity[...] = w.capacity * 8
    w.avail[...] = np.array([[70, 40], [90, 200]], dtype=np.uint16)      # scarce enough that plans change zone and type
    for wl in (w, W.with_bandwidth_polynomials(W.tiny(seed=41, n_types=3, n_zones=2, L=6, p_values=[2, 3, 6]), seed=1)):
        orders = [[0, 1], [1, 0]]
        o = Oracle(wl)
        want = oracle_all(wl, o, orders)
        assert len(want) >= 4
        with Ctx(wl) as cx:
            res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, 32)
        assert_dp_equal(res, st, want, wl, o, orders, 32, wl.name)
        assert any(len(set(x[2]["types"])) > 1 for x in want), "no plan ever mixes types across stages"


def test_dp_eight_types_eight_zones(_index_mode):
    """Eight scarce types in eight zones: one problem's mixed-radix tables need 24 GB, beyond the default
    workspace of 8 GiB; indexed by rank they fit with room to spare."""
    w = W.tiny(seed=14, n_types=8, n_zones=8, L=12, p_values=[12, 5], d_values=(1, 2), tp_values=(1, 2), mbs_values=(1, 4))
    orders = [[7, 6, 5, 4, 3, 2, 1, 0], [2, 5]]
    with Ctx(w) as cx:
        if _index_mode == "dense":
            with pytest.raises(B.SailorError) as e:
                B.sailor_plan_dp(cx.ctx, cx.space, orders, 8)
            assert e.value.code == B.E_RANGE
            return
        o = Oracle(w)
        want = oracle_all(w, o, orders)
        assert len(want) >= 8
        res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, 32)
        assert_dp_equal(res, st, want, w, o, orders, 32, w.name)


@pytest.mark.parametrize("w,orders", list(_tiny()), ids=lambda x: getattr(x, "name", None))
def test_dp_matches_oracle_on_tiny_clusters(w, orders):
    o = Oracle(w)
    want = oracle_all(w, o, orders)
    assert len(want) >= 8
    with Ctx(w) as cx:
        for k in (1, 5, 32):
            res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, k)
            assert_dp_equal(res, st, want, w, o, orders, k, f"{w.name} k={k}")
        # a workspace that forces several batches gives the same answer
        small = max(64 << 10, int(st.workspace_used // 3))
        try:
            res2, st2 = B.sailor_plan_dp(cx.ctx, cx.space, orders, 32, workspace_bytes=small)
        except B.SailorError as e:
            assert e.code == B.E_RANGE                   # one problem alone is larger than a third of the total
        else:
            assert st2.n_batches > 1
            assert_dp_equal(res2, st2, want, w, o, orders, 32, f"{w.name} batched")


@pytest.mark.parametrize("cfg", [1, 2, 6])
def test_dp_matches_oracle_on_workloads(cfg):
    w = W.CONFIGS[cfg]()
    orders = [list(range(w.n_zones))] + ([list(reversed(range(w.n_zones)))] if w.n_zones > 1 else [])
    o = Oracle(w)
    want = oracle_all(w, o, orders)
    with Ctx(w) as cx:
        res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, 16)
        assert_dp_equal(res, st, want, w, o, orders, 16, f"cfg{cfg}")
        # scarce GPUs: counts bind, plans spill into later zones
        avail = (w.avail // 3).astype(np.uint16)
        B.sailor_set_availability(cx.ctx, avail)
        o.set_availability(avail)
        want = oracle_all(w, o, orders)
        res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, 16)
        assert_dp_equal(res, st, want, w, o, orders, 16, f"cfg{cfg} scarce")


def test_dp_sampled_problems_of_the_large_workloads():
    """Workloads 3 and 5: the library solves every problem; the oracle re-solves the winners' problems."""
    for cfg in (3, 5):
        w = W.CONFIGS[cfg]()
        if cfg == 5:                       # the deepest tables of workload 5 run to gigabytes: keep the shallower half
            w.p_values = [p for p in w.p_values if p <= 6]
        orders = [list(range(w.n_zones))]
        o = Oracle(w)
        cfgs = configs_of(w)
        with Ctx(w) as cx:
            res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, 12)
        assert 1 <= len(res) == min(12, st.n_solved)
        assert [(r.value, r.config) for r in res] == sorted((r.value, r.config) for r in res)
        for r in res:
            P, mi, ti, rc, D = cfgs[r.config]
            ref = o.solve_dp(P, mi, ti, rc, D, orders[0])
            assert ref is not None and list(r.type[:P]) == ref["types"] and list(r.zone[:P]) == ref["zones"]
            sim = o.simulate(ref["plan"])
            assert (r.value, r.t_iter, r.cost, r.peak_mem, r.status) == (ref["value"], sim.t_iter, sim.cost, sim.peak_mem, 0)


def test_dp_constraints_drop_plans_after_the_recursion():
    """A budget or a throughput floor is checked on each problem's plan by the simulator's cost and time."""
    w, orders = W.tiny(seed=3, n_types=3, n_zones=2, L=6, p_values=[1, 2, 3, 6]), [[0, 1], [1, 0]]
    o = Oracle(w)
    want = oracle_all(w, o, orders)
    sims = [o.simulate(x[2]["plan"]) for x in want]
    budget = float(np.median([s.cost for s in sims]))
    min_rate = 1.0 / float(np.median([s.t_iter for s in sims]))
    with Ctx(w) as cx:
        for kw in ({"budget": budget}, {"min_rate": min_rate}, {"budget": budget, "min_rate": min_rate}):
            keep = [x for x, s in zip(want, sims)
                    if not (kw.get("budget", 0) > 0 and s.cost > kw["budget"])
                    and not (kw.get("min_rate", 0) > 0 and 1.0 / s.t_iter < kw["min_rate"])]
            assert 0 < len(keep) < len(want)
            res, st = B.sailor_plan_dp(cx.ctx, cx.space, orders, 32, **kw)
            assert st.n_solved == len(want) and st.n_over_constraint == len(want) - len(keep)
            assert [(r.config * len(orders) + r.order) for r in res] == [x[1] for x in keep[:32]]
            assert [r.value for r in res] == [x[0] for x in keep[:32]]


def test_dp_before_any_availability_is_set():
    """A fresh context has no GPUs available on either side: no problem has a plan."""
    w = W.tiny(seed=3)
    ctx = B.sailor_create(w, 0, 0)
    try:
        res, st = B.sailor_plan_dp(ctx, B.make_space(w), [[0, 1]], 4)
        assert res == [] and st.n_solved == 0
    finally:
        B.sailor_destroy(ctx)


def test_dp_argument_checks():
    w = W.tiny(seed=3)
    with Ctx(w) as cx:
        for orders in ([[0, 0]], [[5]], [[]]):
            with pytest.raises(B.SailorError) as e:
                B.sailor_plan_dp(cx.ctx, cx.space, orders, 4)
            assert e.value.code == B.E_ARG
        with pytest.raises(B.SailorError) as e:
            B.sailor_plan_dp(cx.ctx, cx.space, [[0]], 33)
        assert e.value.code == B.E_RANGE
        for obj in (B.Objective(B.OBJ_MIN_COST, 0, 0.0, 0.0, 0.0), B.Objective(B.OBJ_MAX_THROUGHPUT, B.FLAG_EVAL_ALL, 0.0, 0.0, 0.0),
                    B.Objective(B.OBJ_MAX_THROUGHPUT, 0, 0.0, 0.0, 1.2),
                    B.Objective(B.OBJ_MAX_THROUGHPUT, B.DP_FLAG_INDEX_DENSE | B.DP_FLAG_INDEX_COMPACT, 0.0, 0.0, 0.0),
                    B.Objective(B.OBJ_MAX_THROUGHPUT, B.DP_FLAG_ENUM_BY_TYPE | B.DP_FLAG_ENUM_BY_ENTRY, 0.0, 0.0, 0.0)):
            with pytest.raises(B.SailorError) as e:
                B.sailor_plan_dp(cx.ctx, cx.space, [[0]], 4, obj=obj)
            assert e.value.code == B.E_ARG
        with pytest.raises(B.SailorError) as e:
            B.sailor_plan_dp(cx.ctx, cx.space, [[0, 1]], 4, workspace_bytes=64)
        assert e.value.code == B.E_RANGE
        # nothing available: every problem is solved to "no plan"
        B.sailor_set_availability(cx.ctx, np.zeros_like(w.avail))
        res, st = B.sailor_plan_dp(cx.ctx, cx.space, [[0, 1]], 4)
        assert res == [] and st.n_solved == 0
