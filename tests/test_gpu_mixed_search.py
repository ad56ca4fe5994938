"""GPU parity of the search over plans whose stages mix GPU types (Sailor Sec. 4.2.2 "Implementation"):
sailor_plan_mixed, sailor_mixed_decode and sailor_mixed_space_size against the oracle's enumeration and search on
the same seeded inputs.  Flat indices, records, class counts bit-exact; times and costs within 1e-5 relative, and
identical in their bits."""
import ctypes as C

import numpy as np
import pytest

from helpers import REL_TOL_F64, rel_close
from oracle.binding import Oracle
from paper_2504_17096_b200 import binding as B
from paper_2504_17096_b200 import workloads as W

pytestmark = pytest.mark.gpu

COUNT_KEYS = ("n_total", "n_invalid", "n_oom", "n_over_avail", "n_over_constraint", "n_feasible")


@pytest.fixture(scope="module", autouse=True)
def _needs_cuda():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")


class Ctx:
    def __init__(self, w):
        self.ctx = B.sailor_create(w, 0, 0)
        B.sailor_set_availability(self.ctx, w.avail)

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        B.sailor_destroy(self.ctx)


def assert_same(res, st, hits, counts, o, osp, what):
    assert [r.flat for r in res] == [h["flat"] for h in hits], what
    for r, h in zip(res, hits):
        assert r.status == 0 and r.peak_mem == h["peak_mem"], what
        assert rel_close([r.t_iter, r.cost, r.score], [h["t_iter"], h["cost"], h["score"]], REL_TOL_F64), what
        assert (r.t_iter, r.cost, r.score) == (h["t_iter"], h["cost"], h["score"]), what          # identical bits
        assert r.plan.as_dict() == o.mixed_decode(osp, r.flat), what
    assert {k: int(getattr(st, k)) for k in COUNT_KEYS} == {k: counts[k] for k in COUNT_KEYS}, what
    if counts["n_feasible"]:
        assert st.min_feasible_cost == counts["min_cost"], what


def _cases():
    yield W.tiny(seed=3, n_types=2, n_zones=2, L=4, p_values=[1, 2, 4], d_values=(1, 2, 4), seg_max=2), 2, [0, 1]
    yield W.tiny(seed=5, n_types=3, n_zones=1, L=6, p_values=[2, 3], d_values=(4, 6), seg_max=3, gbs=48), 4, [1, 0, 0]
    yield W.tiny(seed=6, n_types=3, n_zones=2, L=4, p_values=[2, 4], d_values=(2, 4), seg_max=2), 4, [0, 0, 1]
    yield W.tiny(seed=11, n_types=4, n_zones=2, L=8, p_values=[3, 8], d_values=(3, 8), seg_max=2, gbs=48), 4, [0, 1, 0, 1]
    deep = W.tiny(seed=13, n_types=3, n_zones=2, L=80, p_values=[5, 40, 80], d_values=(2, 4), seg_max=2, gbs=64)
    deep.avail = deep.avail * 30                      # room for pipelines of 40 and 80 stages (a lane owns two or three)
    deep.name += "-deep"
    yield deep, 2, [0, 0, 1]


@pytest.mark.parametrize("w,gran,tps", list(_cases()), ids=lambda x: getattr(x, "name", None))
def test_mixed_search_matches_oracle(w, gran, tps):
    o = Oracle(w)
    osp = o.mixed_space(gran, tps)
    n = o.mixed_space_size(osp)
    with Ctx(w) as cx:
        sp = B.make_mixed_space(w, gran, tps)
        assert B.sailor_mixed_space_size(cx.ctx, sp) == n
        rng = W.SplitMix64(5)
        for flat in [0, 1, n - 1] + [rng.next_u64() % n for _ in range(200)]:
            assert B.sailor_mixed_decode(cx.ctx, sp, flat).as_dict() == o.mixed_decode(osp, flat)
        with pytest.raises(B.SailorError):
            B.sailor_mixed_decode(cx.ctx, sp, n)
        probe, _ = o.search_mixed(osp, 1, 10_000)
        budget = float(np.median([h["cost"] for h in probe]))
        rate = 1.0 / float(np.median([h["t_iter"] for h in probe]))
        some_mixed = False
        for kind in (0, 1, 2):
            for kw in ({}, {"budget": budget}, {"min_rate": rate}):
                for k in (1, 32):
                    hits, counts = o.search_mixed(osp, kind, k, **kw)
                    obj = B.Objective(kind, 0, kw.get("budget", 0.0), kw.get("min_rate", 0.0), 0.0)
                    res, st = B.sailor_plan_mixed(cx.ctx, sp, obj, k)
                    assert_same(res, st, hits, counts, o, osp, f"{w.name} kind={kind} {kw} k={k}")
                    some_mixed |= any(s.n_groups > 1 for r in res for s in r.plan.stage[: r.plan.P])
        assert some_mixed, "no kept plan ever mixes types inside a stage"


def test_one_part_per_stage_is_the_plain_search():
    """Granularity 1 with one tensor-parallel degree: the space of sailor_plan, index by index."""
    w = W.tiny(seed=9, n_types=3, n_zones=2, L=4, p_values=[1, 2, 4], d_values=(1, 2, 4), tp_values=(1, 2), seg_max=3)
    w.tp_idx = [1]
    with Ctx(w) as cx:
        sp = B.make_mixed_space(w, 1, [1] * w.n_types)
        assert B.sailor_mixed_space_size(cx.ctx, sp) == B.sailor_space_size(cx.ctx, B.make_space(w))
        for kind in (0, 1, 2):
            obj = B.Objective(kind, 0, 0.0, 0.0, 0.0)
            plain, pst = B.sailor_plan(cx.ctx, B.make_space(w), obj, 12)
            mixed, mst = B.sailor_plan_mixed(cx.ctx, sp, obj, 12)
            assert [(r.flat, r.score, r.t_iter, r.cost, r.peak_mem) for r in plain] == \
                   [(r.flat, r.score, r.t_iter, r.cost, r.peak_mem) for r in mixed]
            assert {k: int(getattr(pst, k)) for k in COUNT_KEYS} == {k: int(getattr(mst, k)) for k in COUNT_KEYS}


def test_mixed_search_on_workload_2_with_mixes_beats_or_equals_one_type_per_stage():
    """Workload 2's model and cluster, two pipeline depths: the search over halves and quarters of D contains the
    one-type-per-stage plans of the same tensor-parallel degrees, so its best is at least as good; winners are
    re-simulated by the oracle."""
    w = W.config2()
    w.p_values, w.mbs_idx, w.d_values = [2, 4], [w.mbs_idx[1]], [4, 8]
    tps = [0, 1, 2]
    o = Oracle(w)
    with Ctx(w) as cx:
        obj = B.Objective(0, 0, 0.0, 0.0, 0.0)
        one, _ = B.sailor_plan_mixed(cx.ctx, B.make_mixed_space(w, 1, tps), obj, 8)
        four, st = B.sailor_plan_mixed(cx.ctx, B.make_mixed_space(w, 4, tps), obj, 8)
        assert st.n_total == B.sailor_mixed_space_size(cx.ctx, B.make_mixed_space(w, 4, tps)) and len(four) == 8
        assert four[0].score <= one[0].score
        so, to, co, mo = o.simulate_mixed_batch([r.plan.as_dict() for r in four])
        assert list(so) == [0] * 8 and [r.t_iter for r in four] == list(to) and [r.cost for r in four] == list(co)
        assert [r.peak_mem for r in four] == [int(m) for m in mo]
        assert [(r.score, r.flat) for r in four] == sorted((r.score, r.flat) for r in four)


def test_mixed_search_argument_checks():
    w = W.tiny(seed=3)
    with Ctx(w) as cx:
        sp = B.make_mixed_space(w, 2, [0, 0])
        L = B.load()
        res = (B.MixedResult * 4)()
        n = C.c_uint32()
        ok = B.Objective(0, 0, 0.0, 0.0, 0.0)
        assert L.sailor_plan_mixed(cx.ctx, C.byref(sp), C.byref(ok), 0, res, C.byref(n), None) == B.E_ARG
        assert L.sailor_plan_mixed(cx.ctx, C.byref(sp), C.byref(ok), 33, res, C.byref(n), None) == B.E_RANGE
        for bad in (B.Objective(0, B.FLAG_EVAL_ALL, 0.0, 0.0, 0.0), B.Objective(0, 0, 0.0, 0.0, 1.2)):
            assert L.sailor_plan_mixed(cx.ctx, C.byref(sp), C.byref(bad), 4, res, C.byref(n), None) == B.E_ARG
        deep = B.make_mixed_space(w, 2, [0, 0], p_values=[B.MIX_P_MAX + 1])
        assert L.sailor_plan_mixed(cx.ctx, C.byref(deep), C.byref(ok), 4, res, C.byref(n), None) == B.E_RANGE
        fine = B.make_mixed_space(w, 5, [0, 0], d_values=[17])          # 17 replicas one by one: more units than the limit
        assert L.sailor_plan_mixed(cx.ctx, C.byref(fine), C.byref(ok), 4, res, C.byref(n), None) == B.E_RANGE
        zero = B.make_mixed_space(w, 0, [0, 0])
        assert L.sailor_plan_mixed(cx.ctx, C.byref(zero), C.byref(ok), 4, res, C.byref(n), None) == B.E_ARG
        # nothing available: an empty result, not an error
        B.sailor_set_availability(cx.ctx, np.zeros_like(w.avail))
        none, st = B.sailor_plan_mixed(cx.ctx, sp, ok, 4)
        assert none == [] and st.n_feasible == 0 and st.n_total == B.sailor_mixed_space_size(cx.ctx, sp)
