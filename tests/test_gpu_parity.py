"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Integer results (status, bytes, flat indices, counts) must be bit-exact; times
and costs must agree within 1e-5 relative (binary64) — and, because both sides follow one
written-down operation order without contraction, are also expected to be bit-identical."""
import ctypes as C
import math

import numpy as np
import pytest

from helpers import REL_TOL_F64, golden_cases, rel_close, stages_to_records, workload_from_tables
from oracle.binding import Oracle, parallel_search, plan_snapshots
from paper_2504_17096_b200 import binding as B
from paper_2504_17096_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    return torch


class Ctx:
    def __init__(self, w, avail=None):
        self.w = w
        self.ctx = B.sailor_create(w, 0, 0)
        B.sailor_set_availability(self.ctx, w.avail if avail is None else avail)
        self.space = B.make_space(w)

    def close(self):
        B.sailor_destroy(self.ctx)


@pytest.fixture
def make_ctx(torch_cuda):
    made = []

    def _make(w, avail=None):
        c = Ctx(w, avail)
        made.append(c)
        return c

    yield _make
    for c in made:
        c.close()


def assert_sim_equal(gpu, orc, what=""):
    t, m, c, s = gpu
    so, to, co, mo = orc
    assert np.array_equal(s, so), f"{what}: status differs at {np.flatnonzero(s != so)[:5]}"
    assert np.array_equal(m, mo), f"{what}: peak memory differs at {np.flatnonzero(m != mo)[:5]}"
    assert rel_close(t, to, REL_TOL_F64), f"{what}: t_iter beyond {REL_TOL_F64}"
    assert rel_close(c, co, REL_TOL_F64), f"{what}: cost beyond {REL_TOL_F64}"
    # one operation order on both sides: identical bits
    ok = ~np.isnan(to)
    assert np.array_equal(np.isnan(t), np.isnan(to)) and np.array_equal(np.isnan(c), np.isnan(co))
    assert np.array_equal(t[ok].view(np.uint64), to[ok].view(np.uint64)), f"{what}: t_iter bits"
    assert np.array_equal(c[ok].view(np.uint64), co[ok].view(np.uint64)), f"{what}: cost bits"


# ---- sailor_simulate -----------------------------------------------------------------------------

@pytest.mark.parametrize("case", golden_cases(), ids=lambda c: c["name"])
def test_simulate_hand_worked_cases(case, make_ctx):
    w = workload_from_tables(case["tables"])
    cx = make_ctx(w)
    recs = B.pack_records(stages_to_records([case["plan"]]))
    t, m, c, s = B.sailor_simulate(cx.ctx, recs)
    e = case["expect"]
    assert s[0] == e["status"] and m[0] == e["peak_mem"]
    if e.get("nan"):
        assert math.isnan(t[0]) and math.isnan(c[0])
    else:
        assert t[0] == pytest.approx(e["t_iter"], rel=1e-12)
        assert c[0] == pytest.approx(e["cost"], rel=1e-12)


@pytest.mark.parametrize("cfg", [1, 2, 3, 5])
def test_simulate_random_records_match_oracle(cfg, make_ctx):
    w = W.CONFIGS[cfg]()
    cx = make_ctx(w)
    n = 20011                         # several 256-record tiles and a ragged tail
    recs = W.random_plans(w, n, seed=100 + cfg, hetero_tp=True)
    gpu = B.sailor_simulate(cx.ctx, B.pack_records(recs))
    orc = Oracle(w).simulate_records(recs)
    assert_sim_equal(gpu, orc, f"cfg{cfg}")
    assert len(np.unique(gpu[3])) >= 3          # the sample exercises several status combinations


def test_simulate_tiny_with_latency_terms(make_ctx):
    w = W.tiny(seed=5, n_types=3, n_zones=2)
    cx = make_ctx(w)
    recs = W.random_plans(w, 5000, seed=77, hetero_tp=True)
    assert_sim_equal(B.sailor_simulate(cx.ctx, B.pack_records(recs)), Oracle(w).simulate_records(recs), "tiny")


def test_simulate_device_pointers(make_ctx, torch_cuda):
    torch = torch_cuda
    w = W.config2()
    cx = make_ctx(w)
    n = 4099
    recs = W.random_plans(w, n, seed=9, hetero_tp=False)
    packed = B.pack_records(recs)
    d_plans = torch.from_numpy(packed.view(np.uint8).reshape(n, 72).copy()).cuda()
    t = torch.empty(n, dtype=torch.float64, device="cuda")
    c = torch.empty(n, dtype=torch.float64, device="cuda")
    m = torch.empty(n, dtype=torch.int64, device="cuda")
    s = torch.empty(n, dtype=torch.int32, device="cuda")
    B.sailor_simulate_device(cx.ctx, d_plans.data_ptr(), n, t.data_ptr(), m.data_ptr(), c.data_ptr(), s.data_ptr())
    torch.cuda.synchronize()
    gpu = (t.cpu().numpy(), m.cpu().numpy().view(np.uint64), c.cpu().numpy(), s.cpu().numpy().view(np.uint32))
    assert_sim_equal(gpu, Oracle(w).simulate_records(recs), "device pointers")


def test_simulate_empty_and_bad_records(make_ctx, torch_cuda):
    torch = torch_cuda
    w = W.config1()
    cx = make_ctx(w)
    t, m, c, s = B.sailor_simulate(cx.ctx, np.zeros(0, dtype=B.REC_DTYPE))
    assert t.size == 0
    good = stages_to_records([dict(P=2, mbs_idx=0, rc=0, D=1, type=[0, 1], zone=[0, 0], tp_idx=[0, 0])])
    for field, value in (("P", 3), ("mbs_idx", 9), ("D", 0), ("n_runs", 17)):
        bad = B.pack_records(good)
        bad[field] = value
        with pytest.raises(B.SailorError) as e:
            B.sailor_simulate(cx.ctx, bad)
        assert e.value.code == B.E_RANGE
    bad = B.pack_records(good)
    bad["run"]["type"][0, 1] = 5
    with pytest.raises(B.SailorError):
        B.sailor_simulate(cx.ctx, bad)
    # the same records given on the device are flagged by the kernel's own bounds checks
    both = np.concatenate([B.pack_records(good), bad])
    d = torch.from_numpy(both.view(np.uint8).reshape(2, 72).copy()).cuda()
    st = torch.zeros(2, dtype=torch.int32, device="cuda")
    tt = torch.zeros(2, dtype=torch.float64, device="cuda")
    B.sailor_simulate_device(cx.ctx, d.data_ptr(), 2, tt.data_ptr(), 0, 0, st.data_ptr())
    torch.cuda.synchronize()
    assert st.cpu().tolist()[1] == B.ST_BAD_RECORD and (st.cpu().tolist()[0] & B.ST_BAD_RECORD) == 0
    assert math.isnan(tt.cpu().tolist()[1])
    # a refused device record does not make a later host call fail, and a refused host batch leaves nothing behind
    t, m, c, s = B.sailor_simulate(cx.ctx, B.pack_records(good))
    assert s[0] == Oracle(w).simulate_records(good)[0][0]
    # the host batch with a bad record in it: E_RANGE, results written, the bad one flagged
    L = B.load()
    out_t = np.zeros(2); out_s = np.zeros(2, np.uint32)
    assert L.sailor_simulate(cx.ctx, both.ctypes.data, 2, 0, out_t.ctypes.data, None, None, out_s.ctypes.data) == B.E_RANGE
    assert out_s[1] == B.ST_BAD_RECORD and out_s[0] == s[0] and math.isnan(out_t[1]) and out_t[0] == t[0]
    assert L.sailor_simulate(cx.ctx, both.ctypes.data, 1, 0, out_t.ctypes.data, None, None, out_s.ctypes.data) == B.OK


def test_simulate_host_batch_in_chunks(make_ctx):
    """A host batch larger than what the library stages at a time (chunks of 2^19 records taking turns in three
    slots): every record's results are the oracle's, whichever chunk and slot it went through; a ragged last chunk."""
    w = W.config2()
    cx = make_ctx(w)
    recs = W.random_plans(w, 6007, seed=77, max_runs=8, hetero_tp=True)
    base = B.pack_records(recs)
    n = 4 * (1 << 19) + 200_003                                     # five chunks: slots 0 and 1 are used twice
    big = np.tile(base, n // 6007 + 1)[:n]
    t, m, c, s = B.sailor_simulate(cx.ctx, big)
    so, to, co, mo = Oracle(w).simulate_records(recs)
    idx = np.arange(big.size) % 6007
    assert_sim_equal((t, m, c, s), (so[idx], to[idx], co[idx], mo[idx]), "host batch in chunks")


# ---- enumeration ---------------------------------------------------------------------------------

def _rec_stages(r):
    types, zones, tps = [], [], []
    for q in range(r.n_runs):
        for _ in range(r.run[q].n_stages):
            types.append(r.run[q].type); zones.append(r.run[q].zone); tps.append(r.run[q].tp_idx)
    return (r.P, r.mbs_idx, r.rc, r.D, tuple(types), tuple(zones), tuple(tps))


def _orc_stages(pl):
    return (pl.P, pl.mbs_idx, pl.rc, pl.D, tuple(pl.type[: pl.P]), tuple(pl.zone[: pl.P]), tuple(pl.tp_idx[: pl.P]))


@pytest.mark.parametrize("cfg", [1, 2, 3, 5])
def test_space_size_and_decode_match_oracle(cfg, make_ctx):
    w = W.CONFIGS[cfg]()
    cx = make_ctx(w)
    o = Oracle(w)
    n = B.sailor_space_size(cx.ctx, cx.space)
    assert n == o.space_size() == w.space_size()
    rng = W.SplitMix64(cfg)
    flats = [0, 1, n - 1] + [rng.next_u64() % n for _ in range(300)]
    for f in flats:
        assert _rec_stages(B.sailor_decode(cx.ctx, cx.space, f)) == _orc_stages(o.decode(f))
    with pytest.raises(B.SailorError):
        B.sailor_decode(cx.ctx, cx.space, n)


# ---- sailor_plan ---------------------------------------------------------------------------------

COUNT_KEYS = ("n_total", "n_invalid", "n_oom", "n_over_avail", "n_over_constraint", "n_feasible")


def assert_plan_equal(res, st, hits, counts, oracle, what=""):
    assert [r.flat for r in res] == [h["flat"] for h in hits], what
    for r, h in zip(res, hits):
        assert r.status == 0
        assert r.peak_mem == h["peak_mem"]
        assert rel_close([r.t_iter, r.cost, r.score], [h["t_iter"], h["cost"], h["score"]], REL_TOL_F64)
        assert (r.t_iter, r.cost, r.score) == (h["t_iter"], h["cost"], h["score"])      # identical bits
        assert _rec_stages(r.plan) == _orc_stages(oracle.decode(r.flat))
    if counts is not None:
        assert {k: getattr(st, k) for k in COUNT_KEYS} == {k: counts[k] for k in COUNT_KEYS}, what
        assert st.min_feasible_cost == counts["min_cost"]


@pytest.mark.parametrize("seed,T,Z,seg_max", [(1, 2, 2, 4), (2, 3, 2, 4), (3, 2, 1, 4), (4, 3, 3, 2), (5, 1, 1, 4), (6, 2, 2, 1)])
@pytest.mark.parametrize("objective", [W.OBJ_MAX_THROUGHPUT, W.OBJ_MIN_COST, W.OBJ_MAX_THROUGHPUT_PER_USD])
def test_plan_tiny_spaces_match_exhaustive_oracle(seed, T, Z, seg_max, objective, make_ctx):
    w = W.tiny(seed=seed, n_types=T, n_zones=Z, seg_max=seg_max, objective=objective)
    cx = make_ctx(w)
    o = Oracle(w)
    for k in (1, 7, 32):
        hits, counts = o.search(objective, k)
        for flags in (0, B.FLAG_EVAL_ALL):
            res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=flags), k)
            assert_plan_equal(res, st, hits, counts, o, f"k={k} flags={flags}")


def test_plan_table_limits_64_digits(make_ctx):
    """8 types x 8 zones: 64 digits, the widest mask; two and three segments."""
    for seg_max, p_values, d_values in ((2, [1, 2, 4], (1, 2, 4)), (3, [3, 4], (1, 2))):
        w = W.tiny(seed=20 + seg_max, n_types=8, n_zones=8, seg_max=seg_max, p_values=p_values, d_values=d_values,
                   tp_values=(1, 2), mbs_values=(1, 4), objective=W.OBJ_MAX_THROUGHPUT_PER_USD)
        cx = make_ctx(w)
        o = Oracle(w)
        hits, counts = o.search(w.objective, 32)
        assert counts["n_feasible"] > 32
        for flags in (0, B.FLAG_EVAL_ALL):
            res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=flags), 32)
            assert_plan_equal(res, st, hits, counts, o, f"seg_max={seg_max} flags={flags}")
        n = o.space_size()
        a, b = n // 3 + 5, 2 * n // 3 + 17                       # a range that cuts items in the middle
        hits, counts = o.search(w.objective, 7, lo=a, hi=b)
        res, st = B.sailor_plan_range(cx.ctx, cx.space, B.make_objective(w), a, b, 7)
        assert_plan_equal(res, st, hits, counts, o, "range")


def test_plan_deep_pipelines_up_to_96_stages(make_ctx):
    """The stage limit (96), long runs inside a segment, pipeline depths that do not divide the layer count."""
    w = W.tiny(seed=31, n_types=2, n_zones=2, L=96, p_values=[96, 64, 48, 36, 7], d_values=(1, 2), tp_values=(1, 2),
               mbs_values=(1, 2), gbs=64)
    w.capacity[...] = w.capacity * 8                       # room for 96 layers' worth of state
    w.avail[...] = 400
    cx = make_ctx(w)
    o = Oracle(w)
    for objective in (W.OBJ_MAX_THROUGHPUT, W.OBJ_MIN_COST):
        hits, counts = o.search(objective, 16)
        assert counts["n_feasible"] > 16
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, kind=objective, flags=B.FLAG_EVAL_ALL), 16)
        assert_plan_equal(res, st, hits, counts, o, f"objective {objective}")
    recs = W.random_plans(w, 3000, seed=3, hetero_tp=True)
    assert_sim_equal(B.sailor_simulate(cx.ctx, B.pack_records(recs)), o.simulate_records(recs), "deep")


def test_plan_random_shapes_sweep(make_ctx):
    """Seeded sweep over cluster shapes, layer counts, segment limits, objectives, constraints, k and
    sub-ranges: every search must equal the exhaustive oracle."""
    rng = W.SplitMix64(2024)
    for case in range(24):
        T, Z = rng.randint(1, 4), rng.randint(1, 3)
        L = rng.randint(2, 9)
        seg_max = rng.randint(1, 4)
        objective = rng.randint(0, 2)
        p_values = sorted({rng.randint(1, L) for _ in range(3)})
        w = W.tiny(seed=100 + case, n_types=T, n_zones=Z, L=L, seg_max=seg_max, objective=objective,
                   p_values=p_values, alpha=rng.uniform() * 1e-4)
        if rng.uniform() < 0.3:
            w.has_embed = 0
        if rng.uniform() < 0.3:
            w.has_head = 0
        cx = make_ctx(w)
        o = Oracle(w)
        n = o.space_size()
        k = rng.randint(1, 32)
        kw = {}
        probe, _ = o.search(objective, 32)
        if probe and rng.uniform() < 0.5:
            kw["budget"] = sorted(h["cost"] for h in probe)[len(probe) // 2]
        if probe and rng.uniform() < 0.3:
            kw["min_rate"] = 1.0 / sorted(h["t_iter"] for h in probe)[len(probe) // 2]
        lo, hi = 0, n
        if rng.uniform() < 0.5:
            lo = rng.randint(0, n - 1)
            hi = rng.randint(lo, n)
        flags = B.FLAG_EVAL_ALL if rng.uniform() < 0.5 else 0
        hits, counts = o.search(objective, k, lo=lo, hi=hi, **kw)
        res, st = B.sailor_plan_range(cx.ctx, cx.space, B.make_objective(w, flags=flags, **kw), lo, hi, k)
        assert_plan_equal(res, st, hits, counts, o, f"case {case}: T={T} Z={Z} L={L} seg_max={seg_max} obj={objective} "
                                                    f"P={p_values} k={k} [{lo},{hi}) {kw} flags={flags}")


def test_bandwidth_polynomials_match_oracle(make_ctx):
    """Message-size-dependent bandwidth (Sec. 4.1) in both entry points."""
    for w in (W.with_bandwidth_polynomials(W.tiny(seed=41, n_types=3, n_zones=2), seed=1),
              W.with_bandwidth_polynomials(W.config2(), seed=2)):
        cx = make_ctx(w)
        o = Oracle(w)
        recs = W.random_plans(w, 4000, seed=6, hetero_tp=True)
        assert_sim_equal(B.sailor_simulate(cx.ctx, B.pack_records(recs)), o.simulate_records(recs), w.name)
        hits, counts, budget = o.plan(12)
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w), 12)
        assert_plan_equal(res, st, hits, counts, o, w.name)
    # only some link classes carry a polynomial
    w = W.with_bandwidth_polynomials(W.tiny(seed=42), seed=3)
    w.inter_bw_poly = None
    cx = make_ctx(w)
    o = Oracle(w)
    hits, counts = o.search(w.objective, 8)
    res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w), 8)
    assert_plan_equal(res, st, hits, counts, o, "partial")
    # a polynomial whose constant term is not positive is rejected at create
    w = W.with_bandwidth_polynomials(W.tiny(seed=43), seed=4)
    w.zone_bw_poly[0, 1, 0] = 0.0
    with pytest.raises(B.SailorError) as e:
        B.sailor_create(w, 0, 0)
    assert e.value.code == B.E_ARG


def test_plan_more_stages_than_blocks_and_empty_ranges(make_ctx):
    """Pipelines deeper than the layer count (stages without a block) and empty flat ranges."""
    w = W.tiny(seed=51, n_types=2, n_zones=2, L=2, p_values=[2, 3, 4, 6])
    cx = make_ctx(w)
    o = Oracle(w)
    hits, counts = o.search(w.objective, 10)
    assert counts["n_feasible"] > 0
    for flags in (0, B.FLAG_EVAL_ALL):
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=flags), 10)
        assert_plan_equal(res, st, hits, counts, o, f"flags={flags}")
    recs = W.random_plans(w, 2000, seed=8, hetero_tp=True)
    recs["P"][:50] = 6                                   # force some deep ones (keep run lengths consistent)
    recs["n_runs"][:50] = 1
    recs["n_stages"][:50, 0] = 6
    assert_sim_equal(B.sailor_simulate(cx.ctx, B.pack_records(recs)), o.simulate_records(recs), "deep-short")
    n = o.space_size()
    for lo, hi in ((5, 5), (n, n + 10), (n + 3, n + 1), (7, 3)):
        res, st = B.sailor_plan_range(cx.ctx, cx.space, B.make_objective(w), lo, hi, 4)
        assert res == [] and st.n_total == 0 and st.n_feasible == 0


def test_plan_constraints_and_empty_results(make_ctx):
    w = W.tiny(seed=8, n_types=2, n_zones=2)
    cx = make_ctx(w)
    o = Oracle(w)
    allh, _ = o.search(w.objective, 32)
    budget = sorted(h["cost"] for h in allh)[5]
    rate = 1.0 / allh[10]["t_iter"]
    for kw in (dict(budget=budget), dict(min_rate=rate), dict(budget=budget, min_rate=rate)):
        hits, counts = o.search(w.objective, 9, **kw)
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, **kw), 9)
        assert_plan_equal(res, st, hits, counts, o, str(kw))
    # nothing is available: an empty result, not an error
    B.sailor_set_availability(cx.ctx, np.zeros_like(w.avail))
    res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w), 4)
    assert res == [] and st.n_feasible == 0 and st.n_total == o.space_size()
    # k larger than the feasible set
    B.sailor_set_availability(cx.ctx, w.avail)
    cheap, _ = o.search(W.OBJ_MIN_COST, 6)
    budget = cheap[-1]["cost"]
    hits, counts = o.search(w.objective, 32, budget=budget)
    res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, budget=budget), 32)
    assert 6 <= len(res) == len(hits) < 32
    assert_plan_equal(res, st, hits, counts, o)


def test_plan_argument_errors(make_ctx):
    w = W.tiny(seed=2)
    cx = make_ctx(w)
    L = B.load()
    res = (B.Result * 40)()
    n = C.c_uint32()
    obj = B.make_objective(w)
    assert L.sailor_plan(cx.ctx, C.byref(cx.space), C.byref(obj), 0, res, C.byref(n), None) == B.E_ARG
    assert L.sailor_plan(cx.ctx, C.byref(cx.space), C.byref(obj), 33, res, C.byref(n), None) == B.E_RANGE
    assert L.sailor_plan(cx.ctx, None, C.byref(obj), 1, res, C.byref(n), None) == B.E_ARG
    bad = B.make_space(w)
    bad.n_d = 0
    assert L.sailor_plan(cx.ctx, C.byref(bad), C.byref(obj), 1, res, C.byref(n), None) == B.E_ARG
    bad = B.make_space(w)
    bad.tp_idx[0] = 7
    assert L.sailor_plan(cx.ctx, C.byref(bad), C.byref(obj), 1, res, C.byref(n), None) == B.E_RANGE
    bad = B.make_space(w)
    bad.seg_max = 5
    assert L.sailor_plan(cx.ctx, C.byref(bad), C.byref(obj), 1, res, C.byref(n), None) == B.E_RANGE
    for flags in (16, 0x100, 1 << 31):                   # flags this entry point does not know
        odd = B.make_objective(w, flags=flags)
        assert L.sailor_plan(cx.ctx, C.byref(cx.space), C.byref(odd), 1, res, C.byref(n), None) == B.E_ARG


def test_stats_report_transfer_times_and_launches(make_ctx):
    """One launch per pass (the search kernel's last block merges).  A search carries the snapshot in its launch
    parameters and its kernel writes the results into pinned host memory, so it has no copies of its own to time;
    the device copy of the snapshot that the batch simulator reads is uploaded when that is next called, and its
    device time is then reported."""
    w = W.config2()
    cx = make_ctx(w)
    obj = B.make_objective(w)
    B.sailor_plan(cx.ctx, cx.space, obj, 4)
    B.sailor_set_availability(cx.ctx, w.avail)
    res, st = B.sailor_plan(cx.ctx, cx.space, obj, 4)
    assert st.n_launches == 2 and len(res) == 4           # two passes: cheapest plan, then the budget
    assert st.d2h_ms == 0.0 and 0.0 < st.kernel_ms < 50.0
    res1, st1 = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, factor=0.0), 4)
    assert st1.n_launches == 1
    # the batch simulator reads the snapshot through a pointer: its next call uploads it, the search after reports it
    recs = W.random_plans(w, 100, seed=3)
    half = (w.avail // 2).astype(np.uint16)
    B.sailor_set_availability(cx.ctx, half)
    gpu = B.sailor_simulate(cx.ctx, B.pack_records(recs))
    assert_sim_equal(gpu, Oracle(w, half).simulate_records(recs), "after a new snapshot")
    _, st2 = B.sailor_plan(cx.ctx, cx.space, obj, 4)
    assert 0.0 < st2.h2d_ms < 5.0
    _, st3 = B.sailor_plan(cx.ctx, cx.space, obj, 4)
    assert st3.h2d_ms == st2.h2d_ms                       # no new upload: the last one's time stays


def _same_search(a, b, what):
    (res_a, st_a), (res_b, st_b) = a, b
    assert [(r.flat, r.score, r.t_iter, r.cost, r.peak_mem, r.status) for r in res_a] == \
           [(r.flat, r.score, r.t_iter, r.cost, r.peak_mem, r.status) for r in res_b], what
    assert {k: getattr(st_a, k) for k in COUNT_KEYS} == {k: getattr(st_b, k) for k in COUNT_KEYS}, what
    assert st_a.min_feasible_cost == st_b.min_feasible_cost, what


def test_f32_screen_returns_the_exact_search(make_ctx):
    """SAILOR_FLAG_F32_SCREEN evaluates every candidate in binary32 first and walks an item exactly only when it may
    matter: lists, scores, counts and the cheapest cost must be those of the exact search, bit for bit, and the
    oracle's."""
    rng = W.SplitMix64(77)
    for case in range(10):                                   # tiny spaces against the oracle, all objectives
        T, Z = rng.randint(1, 4), rng.randint(1, 3)
        w = W.tiny(seed=300 + case, n_types=T, n_zones=Z, L=rng.randint(2, 9), seg_max=rng.randint(1, 4),
                   objective=case % 3, alpha=rng.uniform() * 1e-4)
        cx = make_ctx(w)
        o = Oracle(w)
        n = o.space_size()
        k = rng.randint(1, 32)
        lo, hi = (0, n) if case % 2 else (rng.randint(0, n // 2), rng.randint(n // 2, n))
        for extra in (0, B.FLAG_EVAL_ALL):
            hits, counts = o.search(w.objective, k, lo=lo, hi=hi)
            res, st = B.sailor_plan_range(cx.ctx, cx.space, B.make_objective(w, flags=B.FLAG_F32_SCREEN | extra), lo, hi, k)
            assert_plan_equal(res, st, hits, counts, o, f"case {case} flags={extra}")
    for cfg, k in ((1, 32), (6, 16), (3, 16)):               # workloads: against the exact search (itself checked above)
        w = W.CONFIGS[cfg]()
        cx = make_ctx(w)
        kw = dict(budget=0.0, min_rate=0.0, factor=0.0)
        for extra in (0, B.FLAG_EVAL_ALL, B.FLAG_MIN_TP_ONLY):
            exact = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=extra, **kw), k)
            screened = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=extra | B.FLAG_F32_SCREEN, **kw), k)
            _same_search(exact, screened, f"cfg{cfg} flags={extra}")
    w = W.config5()
    cx = make_ctx(w)
    for extra in (0, B.FLAG_EVAL_ALL):
        exact = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=extra), 32)
        screened = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=extra | B.FLAG_F32_SCREEN), 32)
        _same_search(exact, screened, f"cfg5 flags={extra}")
    # the screen is for unconstrained searches
    L = B.load()
    res = (B.Result * 4)()
    nf = C.c_uint32()
    for bad in (B.make_objective(w, flags=B.FLAG_F32_SCREEN, budget=1.0), B.make_objective(w, flags=B.FLAG_F32_SCREEN, min_rate=1.0),
                B.make_objective(w, flags=B.FLAG_F32_SCREEN, factor=1.2), B.make_objective(w, flags=B.FLAG_F32_SCREEN | B.FLAG_DEGREE_ORDER)):
        assert L.sailor_plan(cx.ctx, C.byref(cx.space), C.byref(bad), 4, res, C.byref(nf), None) == B.E_ARG


def test_issue_rate_measurement_is_plausible(torch_cuda):
    """The instruction streams behind the roofline's ceiling: an SM cannot issue more than four warp-instructions
    a cycle, the FP64 pipe runs at about half the FP32 rate, and the streams come close to those limits."""
    r = B.sailor_measure_issue_rates(0, 0, 3)
    props = torch_cuda.cuda.get_device_properties(0)
    limit = props.multi_processor_count * 4 * props.clock_rate * 1e3      # schedulers x max clock
    assert r.sm_count == props.multi_processor_count
    assert 0.5 * limit < r.ffma_warp_inst_per_s <= 1.02 * limit
    assert 0.2 * limit < r.imad_warp_inst_per_s <= 1.02 * limit
    assert 0.2 * limit < r.dadd_warp_inst_per_s <= 0.55 * limit
    assert r.warp_inst_per_run == r.sm_count * 4 * 8 * 2048 * 128


def test_plan_range_split_merges_to_full(make_ctx):
    w = W.config1()
    cx = make_ctx(w)
    o = Oracle(w)
    n = o.space_size()
    obj = B.make_objective(w)
    full, st_full = B.sailor_plan(cx.ctx, cx.space, obj, 16)
    edges = [0, 1, 143, 144, 1000, 3333, 6767, n]
    merged, total = [], 0
    for a, b in zip(edges[:-1], edges[1:]):
        res, st = B.sailor_plan_range(cx.ctx, cx.space, obj, a, b, 16)
        hits, counts = o.search(w.objective, 16, lo=a, hi=b)
        assert_plan_equal(res, st, hits, counts, o, f"[{a},{b})")
        merged += [(r.score, r.flat) for r in res]
        total += st.n_total
    assert total == n == st_full.n_total
    assert sorted(merged)[:16] == [(r.score, r.flat) for r in full]


def test_plan_contexts_with_different_table_sizes_alternate(make_ctx):
    """Two live contexts whose searches need different amounts of shared memory, used in turn."""
    big, small = W.config3(), W.tiny(seed=9, n_types=1, n_zones=1)
    cb, cs = make_ctx(big), make_ctx(small)
    ob = Oracle(small)
    hits, counts = ob.search(small.objective, 4)
    lo, hi = 1000, 200_000
    want, wc = Oracle(big).search(big.objective, 4, lo=lo, hi=hi)
    for _ in range(2):
        res, st = B.sailor_plan_range(cb.ctx, cb.space, B.make_objective(big), lo, hi, 4)
        assert_plan_equal(res, st, want, wc, Oracle(big), "big")
        res, st = B.sailor_plan(cs.ctx, cs.space, B.make_objective(small), 4)
        assert_plan_equal(res, st, hits, counts, ob, "small")


def test_plan_config1_full(make_ctx):
    w = W.config1()
    cx = make_ctx(w)
    o = Oracle(w)
    hits, counts = o.search(w.objective, 32)
    for flags in (0, B.FLAG_EVAL_ALL):
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=flags), 32)
        assert_plan_equal(res, st, hits, counts, o)


def test_plan_config2_budget_factor_two_pass(make_ctx):
    w = W.config2()
    cx = make_ctx(w)
    o = Oracle(w)
    hits, counts, budget = o.plan(16)
    res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w), 16)
    assert st.budget_used == budget
    assert_plan_equal(res, st, hits, counts, o)


def test_plan_config6_min_cost_under_throughput(make_ctx):
    """Minimise cost subject to a minimum throughput (the paper's constrained scenario 1 shape)."""
    w = W.config6()
    cx = make_ctx(w)
    o = Oracle(w)
    hits, counts, _ = o.plan(16)
    assert counts["n_over_constraint"] > 0 and counts["n_feasible"] > 16
    for flags in (0, B.FLAG_EVAL_ALL):
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=flags), 16)
        assert_plan_equal(res, st, hits, counts, o, f"flags={flags}")
    assert all(1.0 / r.t_iter >= w.min_iters_per_s for r in res)


def test_plan_config4_snapshots_replan(make_ctx):
    """Dynamic availability: re-plan per snapshot on one context (only the counts are uploaded); every one
    of the 200 snapshots is compared with the oracle's two-pass plan, and the best plans must all agree."""
    w = W.config4(n_snapshots=200)
    expected = plan_snapshots(w, w.snapshots, 4)         # the oracle, snapshots spread over the host cores
    cx = make_ctx(w)
    o = Oracle(w)
    obj = B.make_objective(w)
    agree = with_plan = 0
    for t, snap in enumerate(w.snapshots):
        hits, counts, budget = expected[t]
        B.sailor_set_availability(cx.ctx, snap)
        res, st = B.sailor_plan(cx.ctx, cx.space, obj, 4)
        if hits:
            with_plan += 1
            assert st.budget_used == budget
            assert_plan_equal(res, st, hits, counts, o, f"snapshot {t}")
            agree += int(res[0].flat == hits[0]["flat"])
        else:
            assert res == []
            agree += 1
    assert agree == 200 and with_plan > 150


def test_plan_config3_full_space(make_ctx):
    """3.6e8 candidates: the whole space on the GPU, the oracle split over the host's cores."""
    w = W.config3()
    cx = make_ctx(w)
    hits, counts = parallel_search(w, w.objective, 16)
    o = Oracle(w)
    for flags in (0, B.FLAG_EVAL_ALL):
        res, st = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w, flags=flags), 16)
        assert_plan_equal(res, st, hits, counts, o, f"flags={flags}")


def test_plan_config5_windows_and_sampled_winner(make_ctx):
    """6.4e9 candidates.  Exact on windows the oracle can enumerate; for the full space the
    winners are re-simulated by the oracle and no sampled candidate may beat them."""
    w = W.config5()
    cx = make_ctx(w)
    o = Oracle(w)
    n = o.space_size()
    obj = B.make_objective(w, flags=B.FLAG_EVAL_ALL)
    rng = W.SplitMix64(55)
    res, st = B.sailor_plan(cx.ctx, cx.space, obj, 32)
    res2, st2 = B.sailor_plan(cx.ctx, cx.space, B.make_objective(w), 32)       # with pruning: same answer
    assert [(r.flat, r.score) for r in res] == [(r.flat, r.score) for r in res2]
    assert {k: getattr(st, k) for k in COUNT_KEYS} == {k: getattr(st2, k) for k in COUNT_KEYS}
    assert st.n_total == n and len(res) == 32 and st.n_feasible > 0
    flats = np.array([r.flat for r in res], dtype=np.uint64)
    so, to, co, mo = o.simulate_flat(flats)
    assert np.all(so == 0)
    assert [r.t_iter for r in res] == list(to) and [r.cost for r in res] == list(co)
    assert [r.peak_mem for r in res] == list(mo)
    assert [(r.score, r.flat) for r in res] == sorted((r.score, r.flat) for r in res)
    # windows the oracle enumerates in full: both ends, random places, and around the winner
    best = int(res[0].flat)
    windows = [(0, 300_000), (n - 250_000, n), (max(0, best - 200_000), min(n, best + 200_000))]
    windows += [(s, s + 400_003) for s in (rng.next_u64() % (n - 500_000) for _ in range(3))]
    for a, b in windows:
        hits, counts = o.search(w.objective, 8, lo=a, hi=b)
        r, s = B.sailor_plan_range(cx.ctx, cx.space, obj, a, b, 8)
        assert_plan_equal(r, s, hits, counts, o, f"[{a},{b})")
    # seeded uniform subsample of 1e6 flat indices: none is feasible and better than the k-th kept
    sample = np.array(sorted({rng.next_u64() % n for _ in range(1_000_000)}), dtype=np.uint64)
    ss, ts, cs_, ms = o.simulate_flat(sample)
    feas = ss == 0
    worst = (res[-1].score, res[-1].flat)
    kept = {r.flat for r in res}
    for f, t in zip(sample[feas], ts[feas]):
        assert (t, int(f)) >= worst or int(f) in kept


def test_config5_sampled_candidates_match_oracle_one_by_one(make_ctx):
    """The seeded uniform subsample of 1e6 flat indices of workload 5, candidate by candidate: the library's
    decoder gives the record, the batch simulator its status, peak bytes, time and cost, and each must equal
    what the oracle computes for the same flat index (integers exact, times and costs identical in their bits)."""
    w = W.config5()
    cx = make_ctx(w)
    o = Oracle(w)
    n = o.space_size()
    rng = W.SplitMix64(55)
    sample = np.array(sorted({rng.next_u64() % n for _ in range(1_000_000)}), dtype=np.uint64)
    recs = (B.PlanRec * sample.size)()
    decode, space = B.load().sailor_decode, C.byref(cx.space)
    for j, f in enumerate(sample.tolist()):
        assert decode(cx.ctx, space, f, C.byref(recs[j])) == 0
    packed = np.frombuffer(recs, dtype=B.REC_DTYPE)
    gpu = B.sailor_simulate(cx.ctx, packed)
    orc = o.simulate_flat(sample)
    assert_sim_equal(gpu, orc, "cfg5 sample")
    # the sample covers every class and every pipeline depth of the space
    assert set(np.unique(packed["P"]).tolist()) == set(w.p_values)
    s = orc[0]
    assert (s == 0).any() and (s & B.ST_OOM).any() and (s & B.ST_OVER_AVAIL).any() and (s & B.ST_INVALID).any()
