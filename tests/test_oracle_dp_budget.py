"""Pins of the oracle's recursion under a cost limit (Sailor Sec. 4.2.3 and the second half of the listing).

Nothing here touches the CUDA library.  The limited recursion is pinned by two cases worked by hand (one in
which checking the limit on the unlimited recursion's plan finds nothing while the limited recursion finds a
plan, one in which a stage is charged a second time with the straggler found behind it), by its reduction to
the unlimited recursion when the limit is infinite, and against brute force over all type sequences with the
charge of Sec. 4.2.3 restated here from per-stage times.
"""
import glob
import itertools
import json
import math
import os

import pytest

from helpers import GOLDEN, workload_from_tables
from oracle.binding import Oracle
from paper_2504_17096_b200 import workloads as W
from test_oracle_dp import _problems, first_fit_zones


def budget_cases():
    out = []
    for path in sorted(glob.glob(os.path.join(GOLDEN, "dp_budget", "*.json"))):
        with open(path) as f:
            out.append(json.load(f))
    return out


@pytest.mark.parametrize("case", budget_cases(), ids=lambda c: c["name"])
def test_hand_worked_limited_recursion(case):
    w = workload_from_tables(case["tables"], case["name"])
    o = Oracle(w)
    p, e = case["problem"], case["expect"]
    args = (p["P"], p["mbs_idx"], p["tp_idx"], p["rc"], p["D"], p["zone_list"])
    r = o.solve_dp_budget(*args, p["limit"])
    assert r["types"] == e["types"] and r["zones"] == e["zones"]
    assert r["value"] == pytest.approx(e["value"], rel=1e-12)
    assert r["charged_cost"] == pytest.approx(e["charged_cost"], rel=1e-12)
    sim = o.simulate(r["plan"])
    assert sim.status == 0 and sim.t_iter == pytest.approx(e["value"], rel=1e-12)
    assert sim.cost == pytest.approx(e["simulated_cost"], rel=1e-12)
    if "unlimited_types" in e:            # the unlimited recursion's plan is over the limit by the simulator's cost
        u = o.solve_dp(*args)
        assert u["types"] == e["unlimited_types"] and u["value"] == pytest.approx(e["unlimited_value"], rel=1e-12)
        assert o.simulate(u["plan"]).cost == pytest.approx(e["unlimited_simulated_cost"], rel=1e-12)
        assert o.simulate(u["plan"]).cost > p["limit"] >= sim.cost
    for other in e.get("other_limits", []):
        q = o.solve_dp_budget(*args, other["limit"])
        assert q["types"] == other["types"] and q["value"] == pytest.approx(other["value"], rel=1e-12)
        assert q["charged_cost"] == pytest.approx(other["charged_cost"], rel=1e-12)
    for limit in e["no_plan_limits"]:
        assert o.solve_dp_budget(*args, limit) is None


def _tiny():
    yield W.tiny(seed=3, n_types=3, n_zones=2, L=6, p_values=[1, 2, 3, 6]), ([0, 1], [1, 0], [1])
    yield W.tiny(seed=7, n_types=2, n_zones=3, L=5, p_values=[2, 4, 5], d_values=(1, 2, 4)), ([0, 1, 2], [2, 0])
    yield W.tiny(seed=8, n_types=4, n_zones=1, L=4, p_values=[1, 3, 4], d_values=(1, 3)), ([0],)


@pytest.mark.parametrize("w,orders", list(_tiny()), ids=lambda x: getattr(x, "name", None))
def test_infinite_limit_is_the_unlimited_recursion(w, orders):
    o = Oracle(w)
    n = 0
    for zone_list in orders:
        for prob in _problems(w):
            a, b = o.solve_dp(*prob, zone_list), o.solve_dp_budget(*prob, zone_list, math.inf)
            assert (a is None) == (b is None)
            if a is not None:
                assert (a["value"], a["types"], a["zones"]) == (b["value"], b["types"], b["zones"])      # identical bits
                n += 1
    assert n > 20


def sequences(w, o, P, mi, ti, rc, D, zone_list):
    """Every type sequence that first fit can place, with its value and its charge by Sec. 4.2.3 restated from
    the simulator's per-stage times: stage j is charged rate_j * N_b * (slowest of stages j..P-1) plus the
    transfer cost of its message when that crosses zones."""
    tp = w.tp_values[ti]
    out = []
    for types in itertools.product(range(w.n_types), repeat=P):
        zones = first_fit_zones(w, w.avail, types, D, tp, zone_list)
        if zones is None:
            continue
        s = o.simulate(o.make_plan(P, mi, rc, D, types, zones, [ti] * P))
        if s.status != 0:
            continue
        t = [s.stage_t[j] for j in range(P)]
        charge = 0.0
        for j in range(P):
            rate = float(D * tp) * (float(w.price_per_hour[zones[j]][types[j]]) / 3600.0)
            charge += rate * (s.n_b * max(t[j:]))
            if j + 1 < P and zones[j] != zones[j + 1]:
                charge += float(2 * s.n_b * D * int(w.p2p_bytes[mi])) * float(w.egress[zones[j]][zones[j + 1]])
        out.append((s.t_iter, charge, list(types)))
    return out


@pytest.mark.parametrize("w,orders", list(_tiny()), ids=lambda x: getattr(x, "name", None))
def test_limited_recursion_against_brute_force(w, orders):
    o = Oracle(w)
    found = none = tight = 0
    for zone_list in orders:
        for prob in _problems(w):
            seqs = sequences(w, o, *prob, zone_list)
            if not seqs:
                assert o.solve_dp_budget(*prob, zone_list, math.inf) is None
                continue
            charges = sorted(c for _, c, _ in seqs)
            P = prob[0]
            # limits between the charges of the sequences (never on one), below the cheapest and above the dearest
            limits = [charges[0] * 0.5, charges[-1] * 2.0] + [0.5 * (a + b) for a, b in zip(charges, charges[1:]) if b > a * (1 + 1e-9)][:6]
            for limit in limits:
                r = o.solve_dp_budget(*prob, zone_list, limit)
                within = [(t, c, ty) for t, c, ty in seqs if c <= limit]
                if r is None:
                    none += 1
                    if P <= 2:               # with at most one choice behind a stage the recursion is exhaustive
                        assert not within
                    continue
                found += 1
                mine = [x for x in seqs if x[2] == r["types"]]
                assert len(mine) == 1
                t_iter, charge, _ = mine[0]
                # the plan is one first fit can place, its charge is the restated one and within the limit, and the
                # simulator reproduces the value from it
                assert r["charged_cost"] == pytest.approx(charge, rel=1e-12) and charge <= limit
                assert r["value"] == pytest.approx(t_iter, rel=1e-12)
                assert r["zones"] == first_fit_zones(w, w.avail, r["types"], prob[4], w.tp_values[prob[2]], zone_list)
                # never better than the best sequence within the limit; equal to it for short pipelines
                best = min(t for t, _, _ in within)
                assert t_iter >= best * (1 - 1e-12)
                if P <= 2:
                    assert t_iter == pytest.approx(best, rel=1e-12)
                tight += len(within) < len(seqs)
    assert found > 50 and none > 5 and tight > 20
