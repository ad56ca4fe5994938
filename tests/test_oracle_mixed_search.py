"""Pins of the oracle's search over plans whose stages mix GPU types (Sailor Sec. 4.2.2 "Implementation": the
resource combinations of a stage).  Nothing here touches the CUDA library.  The combinations are pinned by their
closed-form count and an independent enumeration, the decoder by an independent nested loop, the search by brute
force over plans built here and simulated one by one, and by its reduction to the plain search when a stage may
use one type only."""
import itertools
import math

import pytest

from oracle.binding import Oracle
from paper_2504_17096_b200 import workloads as W


def closed_form(T, units, groups_max=4):
    """Tuples of T non-negative integers adding up to `units` with at most groups_max non-zero entries: choose
    the j non-zero positions, then a composition of `units` into j positive parts."""
    return sum(math.comb(T, j) * math.comb(units - 1, j - 1) for j in range(1, min(groups_max, T, units) + 1))


@pytest.mark.parametrize("T,gran,D", [(1, 4, 8), (2, 4, 8), (3, 4, 4), (3, 4, 6), (4, 2, 2), (6, 4, 8), (8, 4, 16), (5, 3, 7)])
def test_combinations_count_order_and_content(T, gran, D):
    w = W.tiny(seed=2, n_types=T, n_zones=1)
    o = Oracle(w)
    sp = o.mixed_space(gran, [0] * T)
    units = gran if D % gran == 0 else D
    n = o.mixed_n_comb(sp, D)
    assert n == closed_form(T, units)
    mine = sorted((u for u in itertools.product(range(units + 1), repeat=T) if sum(u) == units and sum(x > 0 for x in u) <= 4),
                  reverse=True)
    assert len(mine) == n
    got = [tuple(o.mixed_comb(sp, D, c)) for c in range(n)]
    assert got == mine                                   # descending lexicographic order, nothing missing, nothing twice
    assert got[0] == (units,) + (0,) * (T - 1)
    with pytest.raises(IndexError):
        o.mixed_comb(sp, D, n)


def _space_cases():
    yield W.tiny(seed=3, n_types=2, n_zones=2, L=4, p_values=[1, 2, 4], d_values=(1, 2, 4), seg_max=2), 2, [0, 1]
    yield W.tiny(seed=5, n_types=3, n_zones=1, L=6, p_values=[2, 3], d_values=(4, 6), seg_max=3, gbs=48), 4, [1, 0, 0]
    yield W.tiny(seed=6, n_types=3, n_zones=2, L=4, p_values=[2, 4], d_values=(2, 4), seg_max=2), 4, [0, 0, 1]


@pytest.mark.parametrize("w,gran,tps", list(_space_cases()), ids=lambda x: getattr(x, "name", None))
def test_decode_is_the_nested_enumeration(w, gran, tps):
    o = Oracle(w)
    sp = o.mixed_space(gran, tps)
    n = o.mixed_space_size(sp)
    flat, seen = 0, set()
    for P in w.p_values:                                  # written independently of the flat decoder
        nseg = min(P, w.seg_max)
        for mi in w.mbs_idx:
            for rc in w.rc_values:
                for D in w.d_values:
                    units = gran if D % gran == 0 else D
                    combs = sorted((u for u in itertools.product(range(units + 1), repeat=w.n_types)
                                    if sum(u) == units and sum(x > 0 for x in u) <= 4), reverse=True)
                    digits = [(z, c) for z in range(w.n_zones) for c in range(len(combs))]
                    for segs in itertools.product(digits, repeat=nseg):
                        want = {"P": P, "mbs_idx": mi, "rc": rc, "D": D, "stages": []}
                        for i in range(P):
                            z, c = segs[i * nseg // P]
                            want["stages"].append({"zone": z, "groups": [(g, tps[g], u * (D // units))
                                                                          for g, u in enumerate(combs[c]) if u]})
                        if flat % 7 == 0 or flat < 50:    # every seventh candidate decoded and compared
                            assert o.mixed_decode(sp, flat) == want, flat
                        key = repr(want)
                        assert key not in seen
                        seen.add(key)
                        flat += 1
    assert flat == n
    with pytest.raises(IndexError):
        o.mixed_decode(sp, n)


@pytest.mark.parametrize("w,gran,tps", list(_space_cases()), ids=lambda x: getattr(x, "name", None))
def test_search_against_plans_simulated_one_by_one(w, gran, tps):
    o = Oracle(w)
    sp = o.mixed_space(gran, tps)
    n = o.mixed_space_size(sp)
    rows = []
    for flat in range(n):
        out = o.simulate_mixed(o.mixed_decode(sp, flat))
        rows.append((flat, out.status, out.t_iter, out.cost))
    feasible = [(r[2], r[0]) for r in rows if r[1] == 0]
    assert len(feasible) > 10
    mixed_best = False
    for kind, key in ((0, lambda r: r[2]), (1, lambda r: r[3]), (2, lambda r: r[2] * r[3])):
        budget = sorted(r[3] for r in rows if r[1] == 0)[len(feasible) // 2]
        for kw in ({}, {"budget": budget}):
            ok = [r for r in rows if r[1] == 0 and not (kw and r[3] > budget)]
            want = sorted((key(r), r[0]) for r in ok)[:9]
            hits, counts = o.search_mixed(sp, kind, 9, **kw)
            assert [(h["score"], h["flat"]) for h in hits] == want
            assert counts["n_total"] == n and counts["n_feasible"] == len(ok)
            assert counts["n_invalid"] == sum(1 for r in rows if r[1] & 1)
            assert counts["n_oom"] == sum(1 for r in rows if not r[1] & 1 and r[1] & 4)
            assert counts["n_over_avail"] == sum(1 for r in rows if not r[1] & 5 and r[1] & 2)
            assert counts["n_over_constraint"] == len(feasible) - len(ok)
            best = o.mixed_decode(sp, hits[0]["flat"])
            mixed_best |= any(len(st["groups"]) > 1 for st in best["stages"])
    # sub-ranges add up
    a, _ = o.search_mixed(sp, 0, 5, lo=0, hi=n // 3)
    b, _ = o.search_mixed(sp, 0, 5, lo=n // 3, hi=n)
    full, _ = o.search_mixed(sp, 0, 5)
    assert sorted(a + b, key=lambda h: (h["score"], h["flat"]))[:5] == full


def test_one_part_per_stage_is_the_plain_search():
    """Granularity 1: a stage's replicas all sit on one type, the segment digit becomes zone * T + type, and with one
    tensor-parallel degree the flat order is the plain search's: same candidates, same numbers, same winners."""
    w = W.tiny(seed=9, n_types=3, n_zones=2, L=4, p_values=[1, 2, 4], d_values=(1, 2, 4), tp_values=(1, 2), seg_max=3)
    w.tp_idx = [1]
    o = Oracle(w)
    sp = o.mixed_space(1, [1] * w.n_types)
    assert o.mixed_space_size(sp) == o.space_size()
    for kind in (0, 1, 2):
        plain, pc = o.search(kind, 12)
        mixed, mc = o.search_mixed(sp, kind, 12)
        assert plain == mixed and pc == mc
