"""The allocation-free search entry point against the ordinary one.

`sailor_plan_noalloc` is for callers that must not allocate device memory while they plan (a
process whose memory pool already owns the GPU, a latency-critical re-planning loop that cannot
take cudaMalloc's device-wide stall, a thread running beside a global-mode stream capture).  It
must return exactly what `sailor_plan` returns.  Its working memory is one fixed array shared by
all calls, which still holds the previous call's contents, so every case is run twice in a row,
and with different spaces back to back.  This file sorts last so that it runs after all other
tests; it also passes on its own in a fresh process.
"""
import ctypes as C

import numpy as np
import pytest

from helpers import REL_TOL_F64, rel_close
from paper_2504_17096_b200 import binding as B
from paper_2504_17096_b200 import workloads as W

pytestmark = pytest.mark.gpu

COUNTS = ("n_total", "n_invalid", "n_oom", "n_over_avail", "n_over_constraint", "n_feasible")


def _same(res_a, st_a, res_b, st_b):
    assert [r.flat for r in res_a] == [r.flat for r in res_b]
    for a, b in zip(res_a, res_b):
        assert a.status == b.status and a.peak_mem == b.peak_mem
        assert bytes(a.plan) == bytes(b.plan)
        assert rel_close([a.t_iter, a.cost, a.score], [b.t_iter, b.cost, b.score], REL_TOL_F64)
        assert (a.t_iter, a.cost, a.score) == (b.t_iter, b.cost, b.score)
    assert {k: getattr(st_a, k) for k in COUNTS} == {k: getattr(st_b, k) for k in COUNTS}
    assert st_a.budget_used == st_b.budget_used and st_a.min_feasible_cost == st_b.min_feasible_cost


@pytest.fixture
def contexts():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    made = []

    def make(w):
        ctx = B.sailor_create(w, 0, 0)
        B.sailor_set_availability(ctx, w.avail)
        made.append(ctx)
        return ctx

    yield make
    for ctx in made:
        B.sailor_destroy(ctx)


def test_noalloc_matches_plan_twice_in_a_row(contexts):
    cases = [(W.config2(), 16, 0),                                    # two passes (budget factor), 504 configurations
             (W.tiny(seed=4, n_types=3, n_zones=2, objective=W.OBJ_MIN_COST), 32, B.FLAG_EVAL_ALL),
             (W.config1(), 5, 0)]
    prepared = []
    for w, k, flags in cases:
        ctx = contexts(w)
        space, obj = B.make_space(w), B.make_objective(w, flags=flags)
        want = B.sailor_plan(ctx, space, obj, k)
        assert len(want[0]) > 0
        prepared.append((ctx, space, obj, k, want))
    # the same space twice in a row, then the next space: stale scratch contents must not leak
    for ctx, space, obj, k, want in prepared:
        for _ in range(2):
            got = B.sailor_plan_noalloc(ctx, space, obj, k)
            _same(got[0], got[1], want[0], want[1])
    for ctx, space, obj, k, want in reversed(prepared):
        got = B.sailor_plan_noalloc(ctx, space, obj, k)
        _same(got[0], got[1], want[0], want[1])


def test_noalloc_follows_availability_and_empty_results(contexts):
    w = W.config4(n_snapshots=6)
    ctx = contexts(w)
    space, obj = B.make_space(w), B.make_objective(w)
    for snap in w.snapshots:
        B.sailor_set_availability(ctx, snap)
        want = B.sailor_plan(ctx, space, obj, 4)
        got = B.sailor_plan_noalloc(ctx, space, obj, 4)
        _same(got[0], got[1], want[0], want[1])
    B.sailor_set_availability(ctx, np.zeros_like(w.avail))
    res, st = B.sailor_plan_noalloc(ctx, space, obj, 4)
    assert res == [] and st.n_feasible == 0 and st.n_total == B.sailor_space_size(ctx, space)


def test_noalloc_rejects_spaces_beyond_its_fixed_scratch(contexts):
    w = W.config3()
    ctx = contexts(w)
    space = B.make_space(w)
    obj = B.make_objective(w)
    space.n_d = 32                                    # 10 * 5 * 4 * 2 * 32 = 12 800 configurations > 4096
    for i in range(32):
        space.d_values[i] = 1 << (i % 8)
    res = (B.Result * 4)()
    n = C.c_uint32()
    rc = B.load().sailor_plan_noalloc(ctx, C.byref(space), C.byref(obj), 4, res, C.byref(n), None)
    assert rc == B.E_RANGE
    assert "range" in B.sailor_strerror(rc)
    assert B.load().sailor_plan_noalloc(ctx, C.byref(space), C.byref(obj), 0, res, C.byref(n), None) == B.E_ARG
    # within the limit the same context still works afterwards
    space = B.make_space(w)
    small = B.make_objective(w)
    space.n_p = 3                                     # P in {1, 2, 3}: a few thousand candidates per configuration
    want = B.sailor_plan(ctx, space, small, 8)
    got = B.sailor_plan_noalloc(ctx, space, small, 8)
    _same(got[0], got[1], want[0], want[1])
