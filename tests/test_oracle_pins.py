"""Pins of the CPU oracle against what the paper's formulas and plain mathematics fix.

Nothing here touches the CUDA library.  Hand-worked fixtures, closed forms, invariants and
brute force, chosen so that a dropped term, a wrong index or a transposed table shows.
"""
import copy
import itertools
import math

import numpy as np
import pytest

from helpers import golden_cases, workload_from_tables
from oracle.binding import Oracle, ST_INVALID, ST_OOM, ST_OVER_AVAIL
from paper_2504_17096_b200 import workloads as W

HAND_TOL = 1e-12


@pytest.mark.parametrize("case", golden_cases(), ids=lambda c: c["name"])
def test_hand_worked_cases(case):
    """Sec. 4.3 memory / time / cost formulas on cases worked by hand (tests/golden)."""
    w = workload_from_tables(case["tables"])
    o = Oracle(w)
    p = case["plan"]
    out = o.simulate(o.make_plan(p["P"], p["mbs_idx"], p["rc"], p["D"], p["type"], p["zone"], p["tp_idx"]))
    e = case["expect"]
    assert out.status == e["status"]
    assert out.peak_mem == e["peak_mem"]
    if e.get("nan"):
        assert math.isnan(out.t_iter) and math.isnan(out.cost)
        return
    for key in ("t_iter", "cost", "t_pp", "t_sync", "t_update", "c_comm", "rate_per_s"):
        if key in e:
            assert getattr(out, key) == pytest.approx(e[key], rel=HAND_TOL, abs=1e-18), key
    if "n_b" in e:
        assert out.n_b == e["n_b"]
    for key in ("stage_mem", "stage_t", "stage_sync"):
        if key in e:
            got = list(getattr(out, key)[: p["P"]])
            if key == "stage_mem":
                assert got == e[key]
            else:
                assert got == pytest.approx(e[key], rel=HAND_TOL), key


def _uniform_plan(o, w, P, mbs_idx, tp_idx, D, g, z, rc=0):
    return o.make_plan(P, mbs_idx, rc, D, [g] * P, [z] * P, [tp_idx] * P)


def _strip_embed_head(w):
    w = copy.deepcopy(w)
    w.has_embed = 0
    w.has_head = 0
    return w


def test_homogeneous_closed_form():
    """Sec. 4.2.2 / 4.2.3: identical stages give T_pp = (P + N_b) * t when messages are free."""
    w = _strip_embed_head(W.config1())
    w.intra_inv_bw[...] = 0.0
    w.inter_inv_bw[...] = 0.0
    w.avail[...] = 60000
    o = Oracle(w)
    for P, mi, ti, D, g in itertools.product([1, 2, 4, 8], range(4), range(3), [1, 2, 4], range(2)):
        out = o.simulate(_uniform_plan(o, w, P, mi, ti, D, g, 0))
        n_layers = w.n_blocks // P
        f = sum([w.fwd[W.BLOCK, g, ti, mi]] * n_layers)
        b = sum([w.bwd[W.BLOCK, g, ti, mi]] * n_layers)
        t = f + b
        n_b = w.gbs // (D * w.mbs_values[mi])
        assert out.n_b == n_b
        assert out.t_pp == pytest.approx((P + n_b) * t, rel=1e-13)
        assert out.c_comm == 0.0


def test_homogeneous_with_messages():
    """Same, with a non-zero link: every stage but the last adds two messages."""
    w = _strip_embed_head(W.config1())
    w.avail[...] = 60000
    o = Oracle(w)
    P, mi, ti, D, g = 4, 1, 0, 8, 0      # D*(tp+tp) = 16 > 4 per node -> inter-node link
    out = o.simulate(_uniform_plan(o, w, P, mi, ti, D, g, 0))
    t = 6 * (w.fwd[1, g, ti, mi] + w.bwd[1, g, ti, mi])
    c = float(w.p2p_bytes[mi]) * w.inter_inv_bw[0, g]
    n_b = w.gbs // (D * 2)
    assert out.t_pp == pytest.approx((P * t + (P - 1) * 2 * c) + n_b * (t + 2 * c), rel=1e-13)


def _random_feasible_plans(w, o, n, seed):
    recs = W.random_plans(w, n, seed, hetero_tp=True)
    plans = []
    for j in range(n):
        types, zones, tps = [], [], []
        for r in range(recs["n_runs"][j]):
            for _ in range(recs["n_stages"][j, r]):
                types.append(recs["type"][j, r]); zones.append(recs["zone"][j, r]); tps.append(recs["tp_idx"][j, r])
        pl = o.make_plan(int(recs["P"][j]), int(recs["mbs_idx"][j]), int(recs["rc"][j]), int(recs["D"][j]),
                         types, zones, tps)
        if not (o.simulate(pl).status & ST_INVALID):
            plans.append(pl)
    return plans


@pytest.fixture(scope="module")
def tiny_w():
    return W.tiny(seed=11)


def test_time_monotone_in_bandwidth(tiny_w):
    """Raising any bandwidth (lowering seconds per byte or latency) never raises T_iter."""
    base = Oracle(tiny_w)
    plans = _random_feasible_plans(tiny_w, base, 300, seed=5)
    assert len(plans) > 50
    t0 = [base.simulate(p).t_iter for p in plans]
    strict = 0
    for name in ("intra_inv_bw", "inter_inv_bw", "zone_inv_bw", "intra_alpha", "inter_alpha", "zone_alpha"):
        w2 = copy.deepcopy(tiny_w)
        getattr(w2, name)[...] *= 0.5
        o2 = Oracle(w2)
        t1 = [o2.simulate(p).t_iter for p in plans]
        assert all(b <= a for a, b in zip(t0, t1)), name
        strict += sum(b < a for a, b in zip(t0, t1))
    assert strict > 0


def test_memory_monotone_in_mbs_and_tp(tiny_w):
    """Sec. 4.3: the footprint depends on microbatch size and tp; larger mbs never shrinks it,
    larger tp never grows it (the generated activation tables are monotone)."""
    w = copy.deepcopy(tiny_w)
    w.avail[...] = 60000
    o = Oracle(w)
    for P, D, g, rc in itertools.product([1, 2, 4], [1, 2, 4], range(w.n_types), [0, 1]):
        for ti in range(3):
            mems = [o.simulate(_uniform_plan(o, w, P, mi, ti, D, g, 0, rc)).peak_mem for mi in range(3)]
            # N_b shrinks as mbs grows, so compare only while the in-flight count is capped by P
            if w.gbs // (D * w.mbs_values[2]) >= P:
                assert mems == sorted(mems)
        for mi in range(3):
            mems = [o.simulate(_uniform_plan(o, w, P, mi, ti, D, g, 0, rc)).peak_mem for ti in range(3)]
            assert mems == sorted(mems, reverse=True)


def test_first_stage_holds_most_activations():
    """1F1B: stage i keeps P - i microbatches in flight, so with identical stages M_0 >= M_{P-1}."""
    w = _strip_embed_head(W.tiny(seed=3))
    w.avail[...] = 60000
    o = Oracle(w)
    out = o.simulate(_uniform_plan(o, w, 4, 0, 0, 1, 0, 0))
    mem = list(out.stage_mem[:4])
    assert mem == sorted(mem, reverse=True) and mem[0] > mem[3]
    per_mb = int(w.act_saved[W.BLOCK, 0, 0])
    assert [mem[i] - mem[i + 1] for i in range(3)] == [per_mb] * 3


def test_scaling_invariants(tiny_w):
    """Scaling all times and latencies by a power of two scales T_iter and C_comp exactly and
    leaves C_comm alone; scaling prices scales C_comp only."""
    base = Oracle(tiny_w)
    plans = _random_feasible_plans(tiny_w, base, 200, seed=9)
    ref = [base.simulate(p) for p in plans]
    w2 = copy.deepcopy(tiny_w)
    for name in ("fwd", "bwd", "upd", "intra_alpha", "inter_alpha", "zone_alpha", "intra_inv_bw",
                 "inter_inv_bw", "zone_inv_bw"):
        getattr(w2, name)[...] *= 4.0
    o2 = Oracle(w2)
    for p, r in zip(plans, ref):
        s = o2.simulate(p)
        assert s.t_iter == 4.0 * r.t_iter
        assert s.c_comm == r.c_comm
        assert s.cost - s.c_comm == pytest.approx(4.0 * (r.cost - r.c_comm), rel=1e-12)
        assert s.peak_mem == r.peak_mem and s.status == r.status
    w3 = copy.deepcopy(tiny_w)
    w3.price_per_hour[...] *= 3.0
    o3 = Oracle(w3)
    for p, r in zip(plans, ref):
        s = o3.simulate(p)
        assert s.t_iter == r.t_iter and s.c_comm == r.c_comm
        assert s.cost - s.c_comm == pytest.approx(3.0 * (r.cost - r.c_comm), rel=1e-12)


def test_single_replica_and_single_zone(tiny_w):
    """D = 1 has no gradient synchronisation; a plan inside one zone pays no transfer cost."""
    o = Oracle(tiny_w)
    for pl in _random_feasible_plans(tiny_w, o, 300, seed=13):
        out = o.simulate(pl)
        if pl.D == 1:
            assert out.t_sync == 0.0
        else:
            assert out.t_sync > 0.0
        zones = {pl.zone[i] for i in range(pl.P)}
        if len(zones) == 1:
            assert out.c_comm == 0.0
            assert out.cost == out.rate_per_s * out.t_iter
        crossings = sum(pl.zone[i] != pl.zone[i + 1] for i in range(pl.P - 1))
        assert (out.c_comm > 0.0) == (crossings > 0)


def test_sync_grows_with_d(tiny_w):
    """H3: the all-reduce time grows with the data-parallel degree (once it leaves the node)."""
    w = copy.deepcopy(tiny_w)
    w.avail[...] = 60000
    w.gbs = 48
    o = Oracle(w)
    sync = [o.simulate(_uniform_plan(o, w, 2, 0, 0, D, 0, 0)).t_sync for D in (8, 12, 16, 24, 48)]
    assert sync == sorted(sync) and sync[0] < sync[-1]


def test_memory_mask_independent_of_availability(tiny_w):
    """H2: whether a stage fits in memory does not depend on how many GPUs are available."""
    o = Oracle(tiny_w)
    n = o.space_size()
    flat = np.arange(0, n, 7, dtype=np.uint64)
    st0, _, _, m0 = o.simulate_flat(flat)
    o.set_availability(np.zeros_like(tiny_w.avail))
    st1, _, _, m1 = o.simulate_flat(flat)
    assert np.array_equal(st0 & ST_OOM, st1 & ST_OOM) and np.array_equal(m0, m1)
    assert np.all((st1 & ST_OVER_AVAIL) != 0)


def test_bandwidth_polynomials(tiny_w):
    """Sec. 4.1: bandwidth as a fitted polynomial of the message size.  A constant polynomial equals
    the constant-bandwidth model (up to the rounding of 1/x), and more bandwidth never costs time."""
    base = Oracle(tiny_w)
    plans = _random_feasible_plans(tiny_w, base, 200, seed=17)
    ref = [base.simulate(p) for p in plans]
    w2 = copy.deepcopy(tiny_w)
    const = lambda inv: np.stack([1.0 / inv, 0 * inv, 0 * inv, 0 * inv], axis=-1)
    w2.intra_bw_poly, w2.inter_bw_poly = const(w2.intra_inv_bw), const(w2.inter_inv_bw)
    zi = np.where(w2.zone_inv_bw > 0, w2.zone_inv_bw, 1.0)
    w2.zone_bw_poly = const(zi)
    for name in ("intra_inv_bw", "inter_inv_bw", "zone_inv_bw"):
        getattr(w2, name)[...] = 123.0                      # must be ignored now
    o2 = Oracle(w2)
    for p, r in zip(plans, ref):
        s = o2.simulate(p)
        assert s.t_iter == pytest.approx(r.t_iter, rel=1e-13) and s.cost == pytest.approx(r.cost, rel=1e-13)
        assert s.status == r.status and s.peak_mem == r.peak_mem
    w3 = W.with_bandwidth_polynomials(copy.deepcopy(tiny_w), seed=5)
    o3 = Oracle(w3)
    t3 = [o3.simulate(p).t_iter for p in plans]
    w4 = copy.deepcopy(w3)
    for name in ("intra_bw_poly", "inter_bw_poly", "zone_bw_poly"):
        getattr(w4, name)[...] *= 2.0
    o4 = Oracle(w4)
    t4 = [o4.simulate(p).t_iter for p in plans]
    assert all(b <= a for a, b in zip(t3, t4)) and any(b < a for a, b in zip(t3, t4))
    assert any(abs(a - r.t_iter) > 1e-9 for a, r in zip(t3, ref))      # the curves do change the times


# ---- enumeration -------------------------------------------------------------------------------

def test_space_size_closed_form():
    for cfg, expect in ((1, 6768), (2, 438984), (3, 361094400), (5, 6397205760)):
        w = W.CONFIGS[cfg]()
        assert Oracle(w).space_size() == expect == w.space_size()


def _nested_enumeration(w):
    """Independent of the flat decoder: explicit nested loops, outermost first."""
    T, Z = w.n_types, w.n_zones
    for P in w.p_values:
        nseg = min(P, w.seg_max)
        for mi in w.mbs_idx:
            for ti in w.tp_idx:
                for rc in w.rc_values:
                    for D in w.d_values:
                        for segs in itertools.product(range(T * Z), repeat=nseg):
                            types = [segs[(i * nseg) // P] % T for i in range(P)]
                            zones = [segs[(i * nseg) // P] // T for i in range(P)]
                            yield (P, mi, rc, D, tuple(types), tuple(zones), ti)


def _plan_key(pl):
    return (pl.P, pl.mbs_idx, pl.rc, pl.D, tuple(pl.type[: pl.P]), tuple(pl.zone[: pl.P]), pl.tp_idx[0])


@pytest.mark.parametrize("zones,seg_max", [(1, 4), (2, 4), (2, 2)])
def test_decode_matches_nested_loops(zones, seg_max):
    w = W.tiny(seed=21, n_types=2, n_zones=zones, seg_max=seg_max)
    o = Oracle(w)
    want = list(_nested_enumeration(w))
    assert len(want) == o.space_size()
    got = [_plan_key(o.decode(f)) for f in range(len(want))]
    assert got == want                      # same plans in the same order
    assert len(set(got)) == len(got)        # a bijection
    with pytest.raises(IndexError):
        o.decode(len(want))


def test_decode_is_injective_on_config1():
    w = W.config1()
    o = Oracle(w)
    keys = {_plan_key(o.decode(f)) for f in range(o.space_size())}
    assert len(keys) == 6768


@pytest.mark.parametrize("objective", [W.OBJ_MAX_THROUGHPUT, W.OBJ_MIN_COST, W.OBJ_MAX_THROUGHPUT_PER_USD])
def test_search_equals_brute_force(objective):
    """Sec. 4.2: sort by the objective, return the best — against an explicit sort of every plan."""
    w = W.tiny(seed=33, n_types=2, n_zones=2, objective=objective)
    o = Oracle(w)
    rows = []
    n_inv = n_oom = n_av = 0
    for flat, key in enumerate(_nested_enumeration(w)):
        P, mi, rc, D, types, zones, ti = key
        out = o.simulate(o.make_plan(P, mi, rc, D, types, zones, [ti] * P))
        if out.status & ST_INVALID:
            n_inv += 1
        elif out.status & ST_OOM:
            n_oom += 1
        elif out.status & ST_OVER_AVAIL:
            n_av += 1
        else:
            score = (out.t_iter, out.cost, out.t_iter * out.cost)[objective]
            rows.append((score, flat, out.t_iter, out.cost, out.peak_mem))
    rows.sort()
    assert len(rows) > 20
    hits, counts = o.search(objective, 10)
    assert [(h["score"], h["flat"]) for h in hits] == [r[:2] for r in rows[:10]]
    assert [(h["t_iter"], h["cost"], h["peak_mem"]) for h in hits] == [r[2:] for r in rows[:10]]
    assert counts == dict(n_total=o.space_size(), n_invalid=n_inv, n_oom=n_oom, n_over_avail=n_av,
                          n_over_constraint=0, n_feasible=len(rows), min_cost=min(r[3] for r in rows))
    # k larger than the feasible set returns them all, sorted
    hits_all, _ = o.search(objective, len(rows) + 5)
    assert [h["flat"] for h in hits_all] == [r[1] for r in rows]
    # constraints: budget and minimum throughput only remove plans
    costs = sorted(r[3] for r in rows)
    budget = costs[len(costs) // 3]
    hb, cb = o.search(objective, 5, budget=budget)
    kept = [r for r in rows if r[3] <= budget]
    assert [h["flat"] for h in hb] == [r[1] for r in kept[:5]]
    assert cb["n_feasible"] == len(kept) and cb["n_over_constraint"] == len(rows) - len(kept)
    rate = 1.0 / sorted(r[2] for r in rows)[len(rows) // 2]
    hr, cr = o.search(objective, 5, min_rate=rate)
    kept = [r for r in rows if 1.0 / r[2] >= rate]
    assert [h["flat"] for h in hr] == [r[1] for r in kept[:5]]


def test_range_split_merges_to_the_same_answer():
    from oracle.binding import merge_hits
    w = W.tiny(seed=35)
    o = Oracle(w)
    n = o.space_size()
    full, cf = o.search(w.objective, 8)
    parts = [o.search(w.objective, 8, lo=a, hi=b) for a, b in ((0, n // 3), (n // 3, n // 2), (n // 2, n))]
    assert merge_hits([p[0] for p in parts], 8) == full
    assert sum(p[1]["n_feasible"] for p in parts) == cf["n_feasible"]


def test_budget_factor_two_pass():
    """Max throughput under budget = 1.2 x the cheapest feasible plan (Sec. 5.2.4, scenario 2 shape)."""
    w = W.config2()
    o = Oracle(w)
    cheapest, _ = o.search(W.OBJ_MIN_COST, 1)
    hits, counts, budget = o.plan(4)
    assert budget == 1.2 * cheapest[0]["cost"]
    assert all(h["cost"] <= budget for h in hits)
    unconstrained, _ = o.search(W.OBJ_MAX_THROUGHPUT, 1)
    assert unconstrained[0]["t_iter"] <= hits[0]["t_iter"]
    assert counts["n_over_constraint"] > 0
