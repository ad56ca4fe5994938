"""Pins of the oracle's simulator for plans whose stages mix GPU types among their replicas (Sailor Sec. 4.2
problem statement, Sec. 4.3).  Nothing here touches the CUDA library.

Pinned by a case worked by hand, by the reduction to the plain simulator when no stage mixes, by the
exact identity "two homogeneous pipelines side by side = the slower of the two", and by monotonicity.
"""
import copy
import glob
import json
import math
import os

import numpy as np
import pytest

from helpers import GOLDEN, workload_from_tables
from oracle.binding import Oracle, ST_INVALID, ST_OOM, ST_OVER_AVAIL
from paper_2504_17096_b200 import workloads as W


def mixed_cases():
    out = []
    for path in sorted(glob.glob(os.path.join(GOLDEN, "mixed", "*.json"))):
        with open(path) as f:
            out.append(json.load(f))
    return out


def as_plan(p):
    return {**p, "stages": [{"zone": s["zone"], "groups": [tuple(g) for g in s["groups"]]} for s in p["stages"]]}


@pytest.mark.parametrize("case", mixed_cases(), ids=lambda c: c["name"])
def test_hand_worked_mixed_plan(case):
    o = Oracle(workload_from_tables(case["tables"], case["name"]))
    out = o.simulate_mixed(as_plan(case["plan"]))
    e = case["expect"]
    assert out.status == e["status"] and out.peak_mem == e["peak_mem"] and out.n_b == e["n_b"]
    for key in ("t_iter", "cost", "t_pp", "t_sync", "t_update", "rate_per_s", "c_comm"):
        assert getattr(out, key) == pytest.approx(e[key], rel=1e-12, abs=1e-18), key
    assert list(out.stage_mem[: case["plan"]["P"]]) == e["stage_mem"]


def _same(a, b):
    return a == b or (math.isnan(a) and math.isnan(b))


@pytest.mark.parametrize("w", [W.tiny(seed=3, n_types=3, n_zones=2, L=6, p_values=[1, 2, 3, 6]), W.config2(),
                               W.config5()],                       # the last one with pipelines of up to 96 stages
                         ids=lambda w: w.name)
def test_one_group_per_stage_is_the_plain_simulator(w):
    """No mixing: bit-identical to the simulator for plans whose replicas are all alike."""
    o = Oracle(w)
    rng = W.SplitMix64(77)
    seen, timed, deep = set(), 0, w.n_blocks >= 96
    for _ in range(1500):
        P = rng.randint(1, w.n_blocks) if deep else w.p_values[rng.randint(0, len(w.p_values) - 1)]
        D = w.d_values[rng.randint(0, len(w.d_values) - 1)]
        mi, rc = rng.randint(0, len(w.mbs_values) - 1), w.rc_values[rng.randint(0, len(w.rc_values) - 1)]
        types = [rng.randint(0, w.n_types - 1) for _ in range(P)]
        zones = [rng.randint(0, w.n_zones - 1) for _ in range(P)]
        tps = [rng.randint(0, len(w.tp_values) - 1) for _ in range(P)]
        if rng.uniform() < 0.5:                                    # one kind of stage throughout: these can be feasible when deep
            types, zones, tps = [types[0]] * P, [zones[0]] * P, [tps[0]] * P
        a = o.simulate(o.make_plan(P, mi, rc, D, types, zones, tps))
        b = o.simulate_mixed({"P": P, "mbs_idx": mi, "rc": rc, "D": D,
                              "stages": [{"zone": z, "groups": [(g, t, D)]} for g, z, t in zip(types, zones, tps)]})
        assert (a.status, a.peak_mem, a.n_b) == (b.status, b.peak_mem, b.n_b)
        for key in ("t_iter", "cost", "t_pp", "t_sync", "t_update", "rate_per_s", "c_comm"):
            assert _same(getattr(a, key), getattr(b, key)), key
        seen.add(a.status)
        timed += (not math.isnan(a.t_iter)) and P > 32
    assert (0 in seen or deep) and len(seen) >= 3
    assert timed > 100 or not deep


def test_two_homogeneous_pipelines_side_by_side():
    """Every stage splits D the same way into type a and type b: the pipelines are the all-a and the all-b
    pipeline, and the slower of the two plain results is the answer (messages never stay inside a node here)."""
    w = W.tiny(seed=5, n_types=3, n_zones=2, L=6, p_values=[1, 2, 3, 6])
    w.gpus_per_node[...] = 1
    w.avail[...] = 60000
    o = Oracle(w)
    rng = W.SplitMix64(5)
    checked = 0
    for _ in range(400):
        P = w.p_values[rng.randint(0, len(w.p_values) - 1)]
        D = [2, 3, 4, 8][rng.randint(0, 3)]
        n_a = rng.randint(1, D - 1)
        mi, rc = rng.randint(0, len(w.mbs_values) - 1), rng.randint(0, 1)
        a, b = rng.randint(0, w.n_types - 1), rng.randint(0, w.n_types - 1)
        zones = [rng.randint(0, w.n_zones - 1) for _ in range(P)]
        mixed = o.simulate_mixed({"P": P, "mbs_idx": mi, "rc": rc, "D": D,
                                  "stages": [{"zone": z, "groups": [(a, 0, n_a), (b, 0, D - n_a)]} for z in zones]})
        pa = o.simulate(o.make_plan(P, mi, rc, D, [a] * P, zones, [0] * P))
        pb = o.simulate(o.make_plan(P, mi, rc, D, [b] * P, zones, [0] * P))
        if mixed.status & ST_INVALID:
            assert pa.status & ST_INVALID
            continue
        assert mixed.t_pp == max(pa.t_pp, pb.t_pp)                     # identical bits
        assert mixed.t_update == max(pa.t_update, pb.t_update)
        assert mixed.t_sync == max(pa.t_sync, pb.t_sync)               # D*tp > 1 GPU per node: inter-node in all three
        assert mixed.peak_mem == max(pa.peak_mem, pb.peak_mem)
        assert mixed.c_comm == pa.c_comm == pb.c_comm
        assert mixed.rate_per_s == pytest.approx((n_a * pa.rate_per_s + (D - n_a) * pb.rate_per_s) / D, rel=1e-12)
        checked += 1
    assert checked > 200


def test_replacing_a_replica_by_a_slower_type_never_speeds_up():
    w = W.tiny(seed=6, n_types=3, n_zones=1, L=6, p_values=[2, 3, 6])
    w.avail[...] = 60000
    w.capacity[...] = 1 << 60
    # make type 2 slower than type 0 in every table entry, with the same links
    w.fwd[:, 2] = w.fwd[:, 0] * 1.5
    w.bwd[:, 2] = w.bwd[:, 0] * 1.5
    w.upd[:, 2] = w.upd[:, 0] * 1.5
    for name in ("intra_alpha", "intra_inv_bw", "inter_alpha", "inter_inv_bw"):
        getattr(w, name)[:, 2] = getattr(w, name)[:, 0]
    o = Oracle(w)
    rng = W.SplitMix64(9)
    strict = 0
    for _ in range(300):
        P = w.p_values[rng.randint(0, len(w.p_values) - 1)]
        D = [2, 4, 8][rng.randint(0, 2)]
        mi = rng.randint(0, len(w.mbs_values) - 1)
        base = {"P": P, "mbs_idx": mi, "rc": 0, "D": D, "stages": [{"zone": 0, "groups": [(0, 0, D)]} for _ in range(P)]}
        t0 = o.simulate_mixed(base)
        if t0.status & ST_INVALID:
            continue
        i = rng.randint(0, P - 1)
        n_slow = rng.randint(1, D - 1)
        worse = copy.deepcopy(base)
        worse["stages"][i]["groups"] = [(0, 0, D - n_slow), (2, 0, n_slow)]
        t1 = o.simulate_mixed(worse)
        assert t1.t_iter >= t0.t_iter
        strict += t1.t_iter > t0.t_iter
    assert strict > 50


def test_mixed_status_bits():
    w = W.tiny(seed=3, n_types=2, n_zones=1, L=4, p_values=[2])
    o = Oracle(w)
    ok = {"P": 2, "mbs_idx": 0, "rc": 0, "D": 2, "stages": [{"zone": 0, "groups": [(0, 0, 1), (1, 0, 1)]}] * 2}
    assert o.simulate_mixed(ok).status == 0
    short = copy.deepcopy(ok); short["stages"] = [{"zone": 0, "groups": [(0, 0, 1)]}, ok["stages"][1]]
    assert o.simulate_mixed(short).status & ST_INVALID           # a stage with fewer than D replicas
    w2 = copy.deepcopy(w); w2.avail[0, 1] = 1
    assert Oracle(w2).simulate_mixed(ok).status == ST_OVER_AVAIL  # two stages take one GPU of type 1 each
    w3 = copy.deepcopy(w); w3.capacity[1] = 1
    out = Oracle(w3).simulate_mixed(ok)
    assert out.status == ST_OOM and not math.isnan(out.t_iter)
