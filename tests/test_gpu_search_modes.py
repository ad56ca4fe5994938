"""GPU parity of the pruned search modes (Sailor Sec. 4.2.1: H2 taken to the smallest fitting
tensor-parallel degree, H3/H4 degree order with early termination): sailor_plan with
SAILOR_FLAG_DEGREE_ORDER / SAILOR_FLAG_MIN_TP_ONLY against the oracle's pruned search on the same
seeded inputs.  Flat indices, class counts and skipped counts bit-exact; times and costs within
1e-5 relative, and identical in their bits."""
import glob
import json
import os

import numpy as np
import pytest

from helpers import GOLDEN, REL_TOL_F64, rel_close, workload_from_tables
from oracle.binding import Oracle, PRUNE_D_ORDER, PRUNE_MIN_TP
from paper_2504_17096_b200 import binding as B
from paper_2504_17096_b200 import workloads as W

pytestmark = pytest.mark.gpu

COUNT_KEYS = ("n_total", "n_invalid", "n_oom", "n_pruned_tp", "n_over_avail", "n_over_constraint", "n_feasible",
              "n_skipped", "n_configs", "n_configs_evaluated")


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


def gpu_flags(modes):
    return (B.FLAG_DEGREE_ORDER if modes & PRUNE_D_ORDER else 0) | (B.FLAG_MIN_TP_ONLY if modes & PRUNE_MIN_TP else 0)


def assert_same(res, st, hits, counts, what):
    assert [r.flat for r in res] == [h["flat"] for h in hits], what
    for r, h in zip(res, hits):
        assert r.status == 0 and r.peak_mem == h["peak_mem"], what
        assert rel_close([r.t_iter, r.cost, r.score], [h["t_iter"], h["cost"], h["score"]], REL_TOL_F64), what
        assert (r.t_iter, r.cost, r.score) == (h["t_iter"], h["cost"], h["score"]), what      # identical bits
    got = {k: int(getattr(st, k)) for k in COUNT_KEYS}
    assert got == {k: counts[k] for k in COUNT_KEYS}, what
    if counts["n_feasible"]:
        assert st.min_feasible_cost == counts["min_cost"], what


def search_cases():
    out = []
    for path in sorted(glob.glob(os.path.join(GOLDEN, "search", "*.json"))):
        with open(path) as f:
            out.append(json.load(f))
    return out


@pytest.mark.parametrize("case", search_cases(), ids=lambda c: c["name"])
def test_hand_worked_searches(case):
    w = workload_from_tables(case["tables"], case["name"])
    for key, val in case["space"].items():
        setattr(w, key, val)
    ob = case["objective"]
    with Ctx(w) as cx:
        obj = B.make_objective(w, kind=ob["kind"], budget=ob["budget"], min_rate=ob["min_rate"], factor=0.0,
                               flags=gpu_flags(case["modes"]))
        res, st = B.sailor_plan(cx.ctx, cx.space, obj, case["k"])
    e = case["expect"]
    assert [r.flat for r in res] == [h["flat"] for h in e["hits"]]
    for r, h in zip(res, e["hits"]):
        assert r.t_iter == pytest.approx(h["t_iter"], rel=1e-12)
        if "cost" in h:
            assert r.cost == pytest.approx(h["cost"], rel=1e-12)
    for key in COUNT_KEYS:
        assert int(getattr(st, key)) == e[key], key


def _tiny_workloads():
    yield W.tiny(seed=3)
    yield W.tiny(seed=5, n_types=3, n_zones=1, d_values=(8, 1, 4, 2), objective=W.OBJ_MIN_COST)
    yield W.tiny(seed=9, n_types=2, n_zones=2, L=6, p_values=[1, 2, 3, 6], d_values=(1, 2, 4, 8, 16), gbs=64, seg_max=2)
    yield W.tiny(seed=12, n_types=4, n_zones=2, L=8, p_values=[2, 4, 8], d_values=(1, 2, 4, 8), tp_values=(4, 1, 2),
                 gbs=64, seg_max=3)
    yield W.tiny(seed=13, n_types=8, n_zones=8, seg_max=2, p_values=[1, 2, 4], d_values=(4, 2, 1), tp_values=(1, 2),
                 mbs_values=(1, 4))


@pytest.mark.parametrize("w", list(_tiny_workloads()), ids=lambda w: w.name)
@pytest.mark.parametrize("modes", [PRUNE_D_ORDER, PRUNE_MIN_TP, PRUNE_D_ORDER | PRUNE_MIN_TP])
def test_modes_match_oracle_on_tiny_spaces(w, modes):
    o = Oracle(w)
    probe_t, _ = o.search(0, 10_000)
    probe_c, _ = o.search(1, 10_000)
    min_rate = 1.0 / float(np.median([h["t_iter"] for h in probe_t]))
    budget = float(np.median([h["cost"] for h in probe_c]))
    kinds = (0, 1) if modes & PRUNE_D_ORDER else (0, 1, 2)
    with Ctx(w) as cx:
        for kind in kinds:
            for kw in ({}, {"budget": budget}, {"min_rate": min_rate}):
                for k in (1, 9, 32):
                    hits, counts = o.search_pruned(kind, k, modes, **kw)
                    obj = B.make_objective(w, kind=kind, flags=gpu_flags(modes), factor=0.0,
                                           budget=kw.get("budget", 0.0), min_rate=kw.get("min_rate", 0.0))
                    res, st = B.sailor_plan(cx.ctx, cx.space, obj, k)
                    assert_same(res, st, hits, counts, f"{w.name} modes={modes} kind={kind} {kw} k={k}")
        if modes == PRUNE_MIN_TP:
            # the tensor-parallel rule also applies when nothing is skipped and in a sub-range
            hits, counts = o.search_pruned(0, 8, modes)
            res, st = B.sailor_plan(cx.ctx, cx.space,
                                    B.make_objective(w, kind=0, flags=gpu_flags(modes) | B.FLAG_EVAL_ALL, factor=0.0,
                                                     budget=0.0, min_rate=0.0), 8)
            assert_same(res, st, hits, counts, f"{w.name} eval-all")


def test_modes_with_deep_pipelines_and_bandwidth_polynomials():
    """Up to 96 stages, non-divisor depths, four segments, message-size-dependent links."""
    deep = W.tiny(seed=31, n_types=2, n_zones=2, L=96, p_values=[96, 48, 7], d_values=(4, 1, 2), tp_values=(1, 2, 4),
                  mbs_values=(1, 2), gbs=64)
    deep.capacity[...] = deep.capacity * 4
    deep.avail[...] = 300
    for w in (deep, W.with_bandwidth_polynomials(W.tiny(seed=41, n_types=3, n_zones=2), seed=1)):
        o = Oracle(w)
        with Ctx(w) as cx:
            for modes in (PRUNE_D_ORDER, PRUNE_MIN_TP, PRUNE_D_ORDER | PRUNE_MIN_TP):
                for kind in (0, 1):
                    hits, counts = o.search_pruned(kind, 16, modes)
                    res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, kind=kind, flags=gpu_flags(modes), factor=0.0,
                                                                               budget=0.0, min_rate=0.0), 16)
                    assert_same(res, st, hits, counts, f"{w.name} modes={modes} kind={kind}")


@pytest.mark.parametrize("cfg", [1, 2, 6])
@pytest.mark.parametrize("modes", [PRUNE_D_ORDER, PRUNE_D_ORDER | PRUNE_MIN_TP, PRUNE_MIN_TP])
def test_modes_match_oracle_on_workloads(cfg, modes):
    """Workloads 1, 2 and 6 in full; workload 2 with its two passes (cheapest plan, then the budget)."""
    w = W.CONFIGS[cfg]()
    o = Oracle(w)
    with Ctx(w) as cx:
        budget = w.budget_usd_per_iter
        if w.budget_factor_over_cheapest > 0:
            cheapest, _ = o.search_pruned(W.OBJ_MIN_COST, 1, modes)
            budget = w.budget_factor_over_cheapest * cheapest[0]["cost"]
        hits, counts = o.search_pruned(w.objective, 16, modes, budget=budget, min_rate=w.min_iters_per_s)
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=gpu_flags(modes)), 16)
        assert_same(res, st, hits, counts, f"cfg{cfg} modes={modes}")
        if w.budget_factor_over_cheapest > 0:
            assert st.budget_used == budget
        if modes & PRUNE_D_ORDER:
            assert st.n_skipped > 0


def test_degree_order_on_the_large_workloads_is_consistent():
    """Workloads 3 and 5 are too large for the oracle's pruned search in a test; what must hold at any
    size: the kept plans re-simulate to the same numbers, the counts add up to the space, the result is
    never better than the exhaustive one, and the search is repeatable."""
    for cfg in (3, 5):
        w = W.CONFIGS[cfg]()
        if cfg == 3:
            w.objective = W.OBJ_MAX_THROUGHPUT           # the workload's own objective has no degree-order rule
        o = Oracle(w)
        with Ctx(w) as cx:
            full, st_full = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w), 8)
            obj = B.make_objective(w, flags=B.FLAG_DEGREE_ORDER)
            res, st = B.sailor_plan(cx.ctx, cx.space, obj, 8)
            again, st2 = B.sailor_plan(cx.ctx, cx.space, obj, 8)
            assert [r.flat for r in res] == [r.flat for r in again]
            assert {k: int(getattr(st, k)) for k in COUNT_KEYS} == {k: int(getattr(st2, k)) for k in COUNT_KEYS}
            assert st.n_total + st.n_skipped == st_full.n_total == w.space_size()
            assert st.n_total == st.n_invalid + st.n_oom + st.n_pruned_tp + st.n_over_avail + st.n_over_constraint + st.n_feasible
            assert 0 < st.n_configs_evaluated <= st.n_configs
            if cfg == 3:                                 # workload 5 has no group with a feasible plan at two degrees
                assert st.n_configs_evaluated < st.n_configs and st.n_skipped > 0
            assert (res[0].score, res[0].flat) >= (full[0].score, full[0].flat)
            flats = np.array([r.flat for r in res], dtype=np.uint64)
            so, to, co, mo = o.simulate_flat(flats)
            assert np.all(so == 0)
            assert [r.t_iter for r in res] == list(to) and [r.cost for r in res] == list(co)
            assert [r.peak_mem for r in res] == [int(m) for m in mo]
            assert sorted((r.score, r.flat) for r in res) == [(r.score, r.flat) for r in res]


def test_degree_order_on_a_four_segment_part_of_workload_3():
    """Workload 3's model and cluster (5 zones x 4 types: 20 digits, four segments) with two pipeline depths and
    a thinned configuration list, so that the oracle's pruned search finishes in seconds: degree order for both
    objectives that have one, alone and with the tensor-parallel rule."""
    w = W.config3()
    w.p_values = [4, 8]
    w.mbs_idx = [w.mbs_idx[0], w.mbs_idx[2]]
    w.tp_idx = [w.tp_idx[1], w.tp_idx[3]]
    w.budget_factor_over_cheapest = 0.0
    o = Oracle(w)
    assert w.radix == 20 and w.space_size() == 2 * (2 * 2 * len(w.rc_values) * len(w.d_values)) * 20 ** 4
    with Ctx(w) as cx:
        for kind, modes in ((W.OBJ_MAX_THROUGHPUT, PRUNE_D_ORDER), (W.OBJ_MIN_COST, PRUNE_D_ORDER | PRUNE_MIN_TP)):
            hits, counts = o.search_pruned(kind, 16, modes)
            obj = B.make_objective(w, kind=kind, flags=gpu_flags(modes), factor=0.0, budget=0.0, min_rate=0.0)
            res, st = B.sailor_plan(cx.ctx, cx.space, obj, 16)
            assert_same(res, st, hits, counts, f"cfg3 part kind={kind} modes={modes}")
            assert counts["n_feasible"] > 16 and 0 < counts["n_configs_evaluated"] <= counts["n_configs"]


def test_mode_argument_checks():
    w = W.tiny(seed=3)
    with Ctx(w) as cx:
        n = w.space_size()
        for obj, call in (
                (B.make_objective(w, kind=2, flags=B.FLAG_DEGREE_ORDER), lambda ob: B.sailor_plan(cx.ctx, cx.space, ob, 4)),
                (B.make_objective(w, kind=0, flags=B.FLAG_DEGREE_ORDER | B.FLAG_EVAL_ALL),
                 lambda ob: B.sailor_plan(cx.ctx, cx.space, ob, 4)),
                (B.make_objective(w, kind=0, flags=B.FLAG_DEGREE_ORDER),
                 lambda ob: B.sailor_plan_range(cx.ctx, cx.space, ob, 1, n, 4)),
                (B.make_objective(w, kind=0, flags=B.FLAG_DEGREE_ORDER),
                 lambda ob: B.sailor_plan_noalloc(cx.ctx, cx.space, ob, 4))):
            with pytest.raises(B.SailorError) as e:
                call(obj)
            assert e.value.code == B.E_ARG
        # the whole range spelled out is still the whole space
        res, st = B.sailor_plan_range(cx.ctx, cx.space, B.make_objective(w, kind=0, flags=B.FLAG_DEGREE_ORDER), 0, n, 4)
        hits, counts = Oracle(w).search_pruned(0, 4, PRUNE_D_ORDER)
        assert_same(res, st, hits, counts, "whole range")
