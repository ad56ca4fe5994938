"""Pins of the oracle's dynamic-programming recursion (Sailor Sec. 4.2.2, Eq. 1).

Nothing here touches the CUDA library.  The recursion is an approximation by construction (the rest
of the pipeline is solved on its own), so it is pinned by a case worked by hand in which it provably
misses the optimum, by equality with the plain recursion that remembers nothing, and against brute
force over all type sequences, placed by a first-fit rule restated here and timed by the simulator.
"""
import glob
import itertools
import json
import os

import pytest

from helpers import GOLDEN, workload_from_tables
from oracle.binding import Oracle
from paper_2504_17096_b200 import workloads as W


def first_fit_zones(w, avail, types, D, tp, zone_list):
    """Zones of a type sequence: each stage in the first zone at or after the previous stage's that still
    has D*tp GPUs of its type; None if some stage finds no zone."""
    need = D * tp
    zp, used, zones = 0, {}, []
    for g in types:
        p = zp
        while p < len(zone_list):
            taken = used.get(g, 0) * need if p == zp else 0
            if int(avail[zone_list[p]][g]) >= taken + need:
                break
            p += 1
        if p == len(zone_list):
            return None
        if p != zp:
            used = {}
            zp = p
        used[g] = used.get(g, 0) + 1
        zones.append(zone_list[p])
    return zones


def brute_force(w, o, P, mbs_idx, tp_idx, rc, D, zone_list):
    """Best simulated time over all type sequences placed by first fit: (t_iter, types) or None."""
    best = None
    for types in itertools.product(range(w.n_types), repeat=P):
        zones = first_fit_zones(w, w.avail, types, D, w.tp_values[tp_idx], zone_list)
        if zones is None:
            continue
        out = o.simulate(o.make_plan(P, mbs_idx, rc, D, types, zones, [tp_idx] * P))
        if out.status != 0:
            continue
        if best is None or out.t_iter < best[0]:
            best = (out.t_iter, list(types))
    return best


def dp_cases():
    out = []
    for path in sorted(glob.glob(os.path.join(GOLDEN, "dp", "*.json"))):
        with open(path) as f:
            out.append(json.load(f))
    return out


@pytest.mark.parametrize("case", dp_cases(), ids=lambda c: c["name"])
def test_hand_worked_recursion(case):
    w = workload_from_tables(case["tables"], case["name"])
    o = Oracle(w)
    p, e = case["problem"], case["expect"]
    r = o.solve_dp(p["P"], p["mbs_idx"], p["tp_idx"], p["rc"], p["D"], p["zone_list"])
    assert r["types"] == e["types"] and r["zones"] == e["zones"]
    assert r["value"] == pytest.approx(e["value"], rel=1e-12)
    assert o.simulate(r["plan"]).t_iter == pytest.approx(e["value"], rel=1e-12)
    opt = brute_force(w, o, p["P"], p["mbs_idx"], p["tp_idx"], p["rc"], p["D"], p["zone_list"])
    assert opt[1] == e["optimum_types"] and opt[0] == pytest.approx(e["optimum"], rel=1e-12)
    if "cost" in e:
        assert o.simulate(r["plan"]).cost == pytest.approx(e["cost"], rel=1e-12)
    for zl in e.get("no_plan_zone_lists", []):
        assert o.solve_dp(p["P"], p["mbs_idx"], p["tp_idx"], p["rc"], p["D"], zl) is None


def _problems(w):
    for P in w.p_values:
        for mi in w.mbs_idx:
            for ti in w.tp_idx:
                for rc in w.rc_values:
                    for D in w.d_values:
                        yield P, mi, ti, rc, D


def _tiny():
    yield W.tiny(seed=3, n_types=3, n_zones=2, L=6, p_values=[1, 2, 3, 6]), ([0, 1], [1, 0], [1])
    yield W.tiny(seed=7, n_types=2, n_zones=3, L=5, p_values=[2, 4, 5], d_values=(1, 2, 4)), ([0, 1, 2], [2, 0], [1])
    yield W.tiny(seed=8, n_types=4, n_zones=1, L=4, p_values=[1, 3, 4], d_values=(1, 3)), ([0],)


@pytest.mark.parametrize("w,orders", list(_tiny()), ids=lambda x: getattr(x, "name", None))
def test_recursion_against_brute_force(w, orders):
    o = Oracle(w)
    found = exact = worse = moved = 0
    for zone_list in orders:
        for P, mi, ti, rc, D in _problems(w):
            r = o.solve_dp(P, mi, ti, rc, D, zone_list)
            plain = o.solve_dp(P, mi, ti, rc, D, zone_list, use_memo=False)
            opt = brute_force(w, o, P, mi, ti, rc, D, zone_list)
            assert (r is None) == (opt is None) == (plain is None)
            if r is None:
                continue
            found += 1
            # remembering states changes nothing but the work
            assert (r["value"], r["types"], r["zones"]) == (plain["value"], plain["types"], plain["zones"])
            assert r["n_states"] <= plain["n_states"]
            # the plan obeys first fit and availability, and the simulator reproduces the value from it
            assert r["zones"] == first_fit_zones(w, w.avail, r["types"], D, w.tp_values[ti], zone_list)
            sim = o.simulate(r["plan"])
            assert sim.status == 0
            assert sim.t_iter == pytest.approx(r["value"], rel=1e-12)
            # never better than the optimum over all type sequences; equal when only one choice is left
            assert sim.t_iter >= opt[0] * (1 - 1e-12)
            if P <= 2:
                assert sim.t_iter == pytest.approx(opt[0], rel=1e-12)
            exact += sim.t_iter == pytest.approx(opt[0], rel=1e-12)
            worse += sim.t_iter > opt[0] * (1 + 1e-9)
            moved += len(set(r["zones"])) > 1
    assert found > 20 and exact > 0
    if len(orders[0]) > 1:
        assert moved > 0, "no plan ever left its first zone"


def test_zone_order_matters_and_limits():
    w = W.tiny(seed=3, n_types=3, n_zones=2, L=6, p_values=[6])
    o = Oracle(w)
    a = o.solve_dp(6, 0, 0, 0, 2, [0, 1])
    b = o.solve_dp(6, 0, 0, 0, 2, [1, 0])
    assert a["zones"][0] == 0 and b["zones"][0] == 1
    # a batch size the degrees do not divide, or a degree the heads do not divide: no plan
    assert o.solve_dp(2, 0, 0, 0, 5, [0, 1]) is None
