"""GPU parity of sailor_simulate_mixed (plans whose stages mix GPU types among their replicas; Sailor
Sec. 4.2, Sec. 4.3) against the oracle on the same seeded plans: status and bytes bit-exact, times and
costs within 1e-5 relative and identical in their bits."""
import glob
import json
import math
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

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        B.sailor_destroy(self.ctx)


def assert_equal(gpu, orc, what):
    t, m, c, s = gpu
    so, to, co, mo = orc
    assert np.array_equal(s, so), f"{what}: status differs at {np.flatnonzero(s != so)[:5]}"
    assert np.array_equal(m, mo), f"{what}: peak memory differs at {np.flatnonzero(m != mo)[:5]}"
    assert rel_close(t, to, REL_TOL_F64) and rel_close(c, co, REL_TOL_F64), what
    ok = ~np.isnan(to)
    assert np.array_equal(np.isnan(t), np.isnan(to)) and np.array_equal(np.isnan(c), np.isnan(co)), what
    assert np.array_equal(t[ok].view(np.uint64), to[ok].view(np.uint64)), f"{what}: t_iter bits"
    assert np.array_equal(c[ok].view(np.uint64), co[ok].view(np.uint64)), f"{what}: cost bits"


def test_hand_worked_mixed_plans():
    for path in sorted(glob.glob(os.path.join(GOLDEN, "mixed", "*.json"))):
        with open(path) as f:
            case = json.load(f)
        w = workload_from_tables(case["tables"], case["name"])
        plan = {**case["plan"], "stages": [{"zone": s["zone"], "groups": [tuple(g) for g in s["groups"]]}
                                           for s in case["plan"]["stages"]]}
        with Ctx(w) as cx:
            t, m, c, s = B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans([plan]))
        e = case["expect"]
        assert s[0] == e["status"] and m[0] == e["peak_mem"]
        assert t[0] == pytest.approx(e["t_iter"], rel=1e-12) and c[0] == pytest.approx(e["cost"], rel=1e-12)


@pytest.mark.parametrize("cfg", [1, 2, 3, 5, 6])
def test_random_mixed_plans_match_oracle(cfg):
    w = W.CONFIGS[cfg]()
    n = 6007                              # several blocks and a ragged tail
    plans = W.random_mixed_plans(w, n, seed=300 + cfg)
    with Ctx(w) as cx:
        gpu = B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans(plans))
    assert_equal(gpu, Oracle(w).simulate_mixed_batch(plans), f"cfg{cfg}")
    assert len(np.unique(gpu[3])) >= 3


def test_mixed_tiny_with_latency_polynomials_and_recomputation():
    for w in (W.tiny(seed=5, n_types=3, n_zones=2, L=7, p_values=[1, 2, 3, 7]),
              W.with_bandwidth_polynomials(W.tiny(seed=41, n_types=3, n_zones=2), seed=1),
              W.tiny(seed=21, n_types=8, n_zones=8, L=32, p_values=[32, 16, 5], d_values=(1, 2, 5, 64), gbs=640)):
        plans = W.random_mixed_plans(w, 3000, seed=17)
        with Ctx(w) as cx:
            gpu = B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans(plans))
        assert_equal(gpu, Oracle(w).simulate_mixed_batch(plans), w.name)


@pytest.mark.parametrize("cfg", [0, 5])
def test_deep_mixed_plans_match_oracle(cfg):
    """Plans of up to 96 stages (a lane owns up to three stages): the full records and records cut to the deepest plan."""
    w = W.CONFIGS[cfg]() if cfg else W.tiny(seed=23, n_types=8, n_zones=8, L=96, p_values=[96, 65, 64, 33, 32, 5],
                                            d_values=(1, 2, 5, 64), gbs=640)
    plans = W.random_mixed_plans(w, 4001, seed=500 + cfg, p_max=96)
    depths = [p["P"] for p in plans]
    assert max(depths) > 64 and sum(1 for d in depths if 32 < d <= 64) > 0 and min(depths) <= 32
    orc = Oracle(w).simulate_mixed_batch(plans)
    with Ctx(w) as cx:
        assert_equal(B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans(plans, stages=B.MIX_P_MAX)), orc, f"cfg{cfg} full records")
        assert_equal(B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans(plans)), orc, f"cfg{cfg} cut records")
        # the boundaries of the lane tiles, one plan each
        edge = [p for p in plans if p["P"] in (31, 32, 33, 63, 64, 65, 95, 96)]
        if edge:
            assert_equal(B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans(edge)), Oracle(w).simulate_mixed_batch(edge), "tile edges")


def test_mixed_record_sizes():
    """sailor_simulate_mixed_strided: record sizes it takes, and a plan deeper than its record."""
    import torch
    w = W.config1()
    plans = [p for p in W.random_mixed_plans(w, 800, seed=9) if p["P"] <= 8]
    orc = Oracle(w).simulate_mixed_batch(plans)
    with Ctx(w) as cx:
        for stages in (8, 10, 32, 96):
            assert_equal(B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans(plans, stages=stages)), orc, f"{stages} stages per record")
        L = B.load()
        packed = B.pack_mixed_plans(plans, stages=8)
        out = np.empty(len(plans)); st = np.empty(len(plans), np.uint32)
        for bad_bytes in (0, 24, 28, 36, 1936):
            assert L.sailor_simulate_mixed_strided(cx.ctx, packed.ctypes.data, len(plans), bad_bytes, 0, out.ctypes.data, None, None,
                                                   st.ctypes.data) == B.E_ARG
        deep = packed[:3].copy()
        deep["P"][1] = 9                                 # more stages than the record holds
        with pytest.raises(B.SailorError) as e:
            B.sailor_simulate_mixed(cx.ctx, deep)
        assert e.value.code == B.E_RANGE
        d = torch.from_numpy(deep.view(np.uint8).reshape(3, deep.itemsize).copy()).cuda()
        ds = torch.zeros(3, dtype=torch.int32, device="cuda"); dt = torch.zeros(3, dtype=torch.float64, device="cuda")
        B.sailor_simulate_mixed_device(cx.ctx, d.data_ptr(), 3, dt.data_ptr(), 0, 0, ds.data_ptr(), record_bytes=deep.itemsize)
        torch.cuda.synchronize()
        assert ds.cpu().tolist()[1] == B.ST_BAD_RECORD and ds.cpu().tolist()[0] == int(orc[0][0]) and math.isnan(dt.cpu().tolist()[1])


def test_mixed_host_batch_in_chunks():
    """A host batch of more chunks than staging slots (64 MB of records a chunk, three slots), deep plans among them."""
    w = W.config5()
    plans = W.random_mixed_plans(w, 3001, seed=31, p_max=96)
    base = B.pack_mixed_plans(plans, stages=B.MIX_P_MAX)            # 1 928 B a record: 34 807 records a chunk
    n = 5 * 34_807 + 1_234
    big = np.tile(base, n // 3001 + 1)[:n]
    so, to, co, mo = Oracle(w).simulate_mixed_batch(plans)
    idx = np.arange(n) % 3001
    with Ctx(w) as cx:
        assert_equal(B.sailor_simulate_mixed(cx.ctx, big), (so[idx], to[idx], co[idx], mo[idx]), "mixed host batch in chunks")


def test_mixed_with_one_group_equals_sailor_simulate():
    """No mixing: the same numbers as the run-length records of sailor_simulate."""
    w = W.config2()
    recs = W.random_plans(w, 2000, seed=4, max_runs=8, hetero_tp=True)
    keep = [j for j in range(2000) if recs["P"][j] <= B.MIX_P_MAX]
    plans = []
    for j in keep:
        stages = []
        for r in range(recs["n_runs"][j]):
            for _ in range(recs["n_stages"][j, r]):
                stages.append({"zone": int(recs["zone"][j, r]),
                               "groups": [(int(recs["type"][j, r]), int(recs["tp_idx"][j, r]), int(recs["D"][j]))]})
        plans.append({"P": int(recs["P"][j]), "mbs_idx": int(recs["mbs_idx"][j]), "rc": int(recs["rc"][j]),
                      "D": int(recs["D"][j]), "stages": stages})
    with Ctx(w) as cx:
        t, m, c, s = B.sailor_simulate(cx.ctx, B.pack_records(recs))
        tm, mm, cm, sm = B.sailor_simulate_mixed(cx.ctx, B.pack_mixed_plans(plans))
    keep = np.array(keep)
    assert np.array_equal(s[keep], sm) and np.array_equal(m[keep], mm)
    ok = ~np.isnan(tm)
    assert np.array_equal(t[keep][ok].view(np.uint64), tm[ok].view(np.uint64))
    assert np.array_equal(c[keep][ok].view(np.uint64), cm[ok].view(np.uint64))


def test_mixed_device_pointers_empty_and_bad_records():
    import torch
    w = W.config1()
    plans = W.random_mixed_plans(w, 1500, seed=8)
    packed = B.pack_mixed_plans(plans)
    with Ctx(w) as cx:
        t, m, c, s = B.sailor_simulate_mixed(cx.ctx, np.zeros(0, dtype=B.MIX_DTYPE))
        assert t.size == 0
        n = packed.size
        d = torch.from_numpy(packed.view(np.uint8).reshape(n, packed.itemsize).copy()).cuda()
        dt = torch.empty(n, dtype=torch.float64, device="cuda"); dc = torch.empty(n, dtype=torch.float64, device="cuda")
        dm = torch.empty(n, dtype=torch.int64, device="cuda"); ds = torch.empty(n, dtype=torch.int32, device="cuda")
        B.sailor_simulate_mixed_device(cx.ctx, d.data_ptr(), n, dt.data_ptr(), dm.data_ptr(), dc.data_ptr(), ds.data_ptr(),
                                       record_bytes=packed.itemsize)
        torch.cuda.synchronize()
        gpu = (dt.cpu().numpy(), dm.cpu().numpy().view(np.uint64), dc.cpu().numpy(), ds.cpu().numpy().view(np.uint32))
        assert_equal(gpu, Oracle(w).simulate_mixed_batch(plans), "device pointers")
        # host records with an index outside its table are refused; on the device the kernel flags them
        bad = packed[:2].copy()
        bad["stage"]["group"]["type"][1, 0, 0] = 7
        with pytest.raises(B.SailorError) as e:
            B.sailor_simulate_mixed(cx.ctx, bad)
        assert e.value.code == B.E_RANGE
        d2 = torch.from_numpy(bad.view(np.uint8).reshape(2, bad.itemsize).copy()).cuda()
        st = torch.zeros(2, dtype=torch.int32, device="cuda"); tt = torch.zeros(2, dtype=torch.float64, device="cuda")
        B.sailor_simulate_mixed_device(cx.ctx, d2.data_ptr(), 2, tt.data_ptr(), 0, 0, st.data_ptr(), record_bytes=bad.itemsize)
        torch.cuda.synchronize()
        assert st.cpu().tolist()[1] == B.ST_BAD_RECORD and not (st.cpu().tolist()[0] & B.ST_BAD_RECORD)
        assert math.isnan(tt.cpu().tolist()[1])
