"""Pins of the oracle's pruned search modes (Sailor Sec. 4.2.1: H2, H3, H4).

Nothing here touches the CUDA library.  The rules are pinned by searches worked by hand
(tests/golden/search), by equality with the exhaustive search when no mode is on, and by a
restatement over per-candidate results that shares no loop with the oracle's search: every
candidate is simulated through its flat index, grouped with numpy, and the modes are applied to
those arrays.
"""
import glob
import json
import os

import numpy as np
import pytest

from helpers import GOLDEN, workload_from_tables
from oracle.binding import Oracle, PRUNE_D_ORDER, PRUNE_MIN_TP, ST_INVALID, ST_OOM, ST_OVER_AVAIL
from paper_2504_17096_b200 import workloads as W

HAND_TOL = 1e-12


def search_cases():
    out = []
    for path in sorted(glob.glob(os.path.join(GOLDEN, "search", "*.json"))):
        with open(path) as f:
            out.append(json.load(f))
    return out


def workload_of_case(case):
    w = workload_from_tables(case["tables"], case["name"])
    for key, val in case["space"].items():
        setattr(w, key, val)
    w.objective = case["objective"]["kind"]
    w.budget_usd_per_iter = case["objective"]["budget"]
    w.min_iters_per_s = case["objective"]["min_rate"]
    return w


@pytest.mark.parametrize("case", search_cases(), ids=lambda c: c["name"])
def test_hand_worked_searches(case):
    w = workload_of_case(case)
    o = Oracle(w)
    ob = case["objective"]
    hits, counts = o.search_pruned(ob["kind"], case["k"], case["modes"], budget=ob["budget"], min_rate=ob["min_rate"])
    e = case["expect"]
    assert [h["flat"] for h in hits] == [h["flat"] for h in e["hits"]]
    for got, want in zip(hits, e["hits"]):
        assert got["t_iter"] == pytest.approx(want["t_iter"], rel=HAND_TOL)
        if "cost" in want:
            assert got["cost"] == pytest.approx(want["cost"], rel=HAND_TOL)
    for key in ("n_total", "n_invalid", "n_oom", "n_pruned_tp", "n_over_avail", "n_over_constraint", "n_feasible",
                "n_skipped", "n_configs", "n_configs_evaluated"):
        assert counts[key] == e[key], key


def _tiny_workloads():
    yield W.tiny(seed=3)
    yield W.tiny(seed=5, n_types=3, n_zones=1, d_values=(8, 1, 4, 2), objective=W.OBJ_MIN_COST)
    yield W.tiny(seed=9, n_types=2, n_zones=2, L=6, p_values=[1, 2, 3, 6], d_values=(1, 2, 4, 8, 16), gbs=64, seg_max=2)


@pytest.mark.parametrize("w", list(_tiny_workloads()), ids=lambda w: w.name)
def test_no_mode_is_the_exhaustive_search(w):
    o = Oracle(w)
    for kind in (0, 1, 2):
        a, ca = o.search(kind, 16)
        b, cb = o.search_pruned(kind, 16, 0)
        assert a == b
        for key in ca:
            assert ca[key] == cb[key], key
        assert cb["n_skipped"] == 0 and cb["n_pruned_tp"] == 0 and cb["n_configs"] == cb["n_configs_evaluated"]


class Table:
    """Every candidate of a space simulated through its flat index, with its digits."""

    def __init__(self, w, o, kind, budget=0.0, min_rate=0.0):
        n = o.space_size()
        self.flat = np.arange(n, dtype=np.uint64)
        st, t, c, _ = o.simulate_flat(self.flat)
        self.st, self.t, self.c = st, t, c
        self.score = {0: t, 1: c, 2: t * c}[kind]
        # digits of every flat index from the documented order: sub-spaces of P one after the other; inside,
        # from the lowest: the segment digits, D, rc, tp, mbs
        base = len(w.mbs_idx) * len(w.tp_idx) * len(w.rc_values) * len(w.d_values)
        self.p = np.zeros(n, np.int64); self.seg = np.zeros(n, np.int64)
        self.di = np.zeros(n, np.int64); self.ri = np.zeros(n, np.int64)
        self.ti = np.zeros(n, np.int64); self.mi = np.zeros(n, np.int64)
        at = 0
        for jp, P in enumerate(w.p_values):
            per = w.radix ** min(P, w.seg_max)
            m = base * per
            x = np.arange(m, dtype=np.int64)
            sl = slice(at, at + m)
            self.p[sl] = jp
            self.seg[sl] = x % per; x //= per
            self.di[sl] = x % len(w.d_values); x //= len(w.d_values)
            self.ri[sl] = x % len(w.rc_values); x //= len(w.rc_values)
            self.ti[sl] = x % len(w.tp_idx); x //= len(w.tp_idx)
            self.mi[sl] = x
            at += m
        over = np.zeros(n, bool)
        with np.errstate(divide="ignore", invalid="ignore"):
            if budget > 0:
                over |= c > budget
            if min_rate > 0:
                over |= 1.0 / t < min_rate
        self.over = over


def _restate(w, o, kind, modes, k, budget=0.0, min_rate=0.0):
    """The modes applied to the per-candidate table: returns (hit flats, counts)."""
    tb = Table(w, o, kind, budget, min_rate)
    invalid = (tb.st & ST_INVALID) != 0
    oom = ~invalid & ((tb.st & ST_OOM) != 0)
    alive = ~invalid & ~oom
    pruned = np.zeros_like(alive)
    if modes & PRUNE_MIN_TP:
        # among the candidates that differ only in tp, keep the smallest tp value that is valid and fits
        tpv = np.array([w.tp_values[j] for j in w.tp_idx], dtype=np.int64)[tb.ti]
        key = ((tb.p * 64 + tb.mi) * 64 + tb.ri) * 64 + tb.di
        key = key * (w.radix ** w.seg_max) + tb.seg
        best_tp = {}
        for kk, v in zip(key[alive], tpv[alive]):
            best_tp[kk] = min(best_tp.get(kk, 1 << 30), v)
        keep = np.array([best_tp.get(kk, -1) == v for kk, v in zip(key, tpv)])
        pruned = alive & ~keep
    rest = alive & ~pruned
    over_avail = rest & ((tb.st & ST_OVER_AVAIL) != 0)
    rest = rest & ~over_avail
    over_c = rest & tb.over
    feas = rest & ~over_c
    cfg = ((tb.p * 64 + tb.mi) * 64 + tb.ti) * 64 + tb.ri
    looked = np.ones_like(alive)
    if modes & PRUNE_D_ORDER:
        looked[:] = False
        dv = np.array(w.d_values)
        order = sorted(range(len(dv)), key=lambda j: (-dv[j] if kind == 0 else dv[j], j))
        for g in np.unique(cfg):
            in_g = cfg == g
            prev = None
            for di in order:
                sel = in_g & (tb.di == di)
                looked |= sel
                f = sel & feas
                if not f.any():
                    if prev is not None:
                        break
                    continue
                best = tb.score[f].min()
                if prev is not None and not best < prev:
                    break
                prev = best
    cand = np.flatnonzero(feas & looked)
    order = sorted(cand, key=lambda j: (tb.score[j], j))[:k]
    counts = {"n_total": int(looked.sum()), "n_invalid": int((invalid & looked).sum()), "n_oom": int((oom & looked).sum()),
              "n_pruned_tp": int((pruned & looked).sum()), "n_over_avail": int((over_avail & looked).sum()),
              "n_over_constraint": int((over_c & looked).sum()), "n_feasible": int((feas & looked).sum()),
              "n_skipped": int((~looked).sum())}
    return [int(j) for j in order], [float(tb.score[j]) for j in order], counts


@pytest.mark.parametrize("w", list(_tiny_workloads()), ids=lambda w: w.name)
@pytest.mark.parametrize("modes", [PRUNE_D_ORDER, PRUNE_MIN_TP, PRUNE_D_ORDER | PRUNE_MIN_TP])
def test_modes_against_the_restatement(w, modes):
    o = Oracle(w)
    seen_skip = False
    for kind, budget, min_rate in ((0, 0.0, 0.0), (1, 0.0, 0.0), (1, 0.0, None), (0, None, 0.0)):
        if min_rate is None:          # a throughput floor that about half of the feasible plans meet
            hits, _ = o.search(0, 10_000)
            min_rate = 1.0 / float(np.median([h["t_iter"] for h in hits]))
        if budget is None:
            hits, _ = o.search(1, 10_000)
            budget = float(np.median([h["cost"] for h in hits]))
        got, counts = o.search_pruned(kind, 12, modes, budget=budget, min_rate=min_rate)
        flats, scores, want = _restate(w, o, kind, modes, 12, budget, min_rate)
        assert [h["flat"] for h in got] == flats
        assert [h["score"] for h in got] == scores
        for key, v in want.items():
            assert counts[key] == v, key
        assert counts["n_total"] + counts["n_skipped"] == o.space_size()
        seen_skip |= counts["n_skipped"] > 0
        # never better than the exhaustive search, and every kept plan is one of its feasible plans
        full, _ = o.search(kind, 1, budget=budget, min_rate=min_rate)
        if got:
            assert (got[0]["score"], got[0]["flat"]) >= (full[0]["score"], full[0]["flat"])
    if modes & PRUNE_D_ORDER:
        assert seen_skip, "the case never exercises early termination"


def test_degree_order_rejects_other_objectives():
    o = Oracle(W.tiny(seed=3))
    with pytest.raises(ValueError):
        o.search_pruned(2, 4, PRUNE_D_ORDER)
    o.search_pruned(2, 4, PRUNE_MIN_TP)      # the tensor-parallel rule does not depend on the objective


def test_single_degree_makes_the_order_irrelevant():
    w = W.tiny(seed=4, d_values=(2,))
    o = Oracle(w)
    a, ca = o.search(0, 8)
    b, cb = o.search_pruned(0, 8, PRUNE_D_ORDER)
    assert a == b and cb["n_skipped"] == 0 and ca["n_feasible"] == cb["n_feasible"]
