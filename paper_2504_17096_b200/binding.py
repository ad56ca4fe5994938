"""ctypes binding of the C ABI in include/sailor.h: the same entry points, arguments marshalled
from numpy arrays / raw device pointers.  No step of the simulation runs here, and there is no
fallback: if the CUDA library is missing, loading it fails loudly."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsailor_b200.so")

KINDS, T_MAX, Z_MAX, TP_MAX, MBS_MAX, P_MAX, RUN_MAX, SEG_MAX, K_MAX, NP_MAX, ND_MAX = 3, 8, 8, 8, 16, 96, 16, 4, 32, 32, 32
OK, E_ARG, E_RANGE, E_CUDA, E_NOMEM, E_DEVICE = 0, -1, -2, -3, -4, -5
ST_INVALID, ST_OVER_AVAIL, ST_OOM, ST_BAD_RECORD = 1, 2, 4, 32
OBJ_MAX_THROUGHPUT, OBJ_MIN_COST, OBJ_MAX_THROUGHPUT_PER_USD = 0, 1, 2
FLAG_EVAL_ALL, FLAG_DEGREE_ORDER, FLAG_MIN_TP_ONLY, FLAG_F32_SCREEN = 1, 2, 4, 8
DP_FLAG_INDEX_DENSE, DP_FLAG_INDEX_COMPACT, DP_FLAG_ENUM_BY_TYPE, DP_FLAG_ENUM_BY_ENTRY = 0x100, 0x200, 0x400, 0x800
DP_FLAG_BUDGET_LOOP, DP_BUDGET_P_MAX = 0x1000, 32

EXPORTS = ("sailor_create", "sailor_destroy", "sailor_set_availability", "sailor_simulate",
           "sailor_space_size", "sailor_decode", "sailor_plan", "sailor_plan_range", "sailor_plan_noalloc",
           "sailor_plan_dp", "sailor_simulate_mixed", "sailor_simulate_mixed_strided", "sailor_mixed_space_size", "sailor_mixed_decode",
           "sailor_plan_mixed", "sailor_measure_issue_rates", "sailor_strerror",
           "sailor_last_cuda_error")

_dp, _u64p, _u32p, _u16p = C.POINTER(C.c_double), C.POINTER(C.c_uint64), C.POINTER(C.c_uint32), C.POINTER(C.c_uint16)


class Model(C.Structure):
    _fields_ = [("n_blocks", C.c_uint32), ("has_embed", C.c_uint32), ("has_head", C.c_uint32), ("heads", C.c_uint32),
                ("gbs", C.c_uint64), ("mul_factor", C.c_uint32), ("dtype_size", C.c_uint32),
                ("grad_dtype_size", C.c_uint32), ("_pad", C.c_uint32)]


class Profile(C.Structure):
    _fields_ = [("n_types", C.c_uint32), ("n_tp", C.c_uint32), ("n_mbs", C.c_uint32), ("_pad", C.c_uint32),
                ("tp_values", C.c_uint32 * TP_MAX), ("mbs_values", C.c_uint32 * MBS_MAX),
                ("fwd", _dp), ("bwd", _dp), ("upd", _dp), ("params", _u64p), ("act_saved", _u64p),
                ("act_ckpt", _u64p), ("act_work", _u64p), ("p2p_bytes", _u64p)]


class Cluster(C.Structure):
    _fields_ = [("n_types", C.c_uint32), ("n_zones", C.c_uint32), ("capacity", _u64p), ("reserved", _u64p),
                ("gpus_per_node", _u32p), ("price_per_hour", _dp), ("intra_alpha", _dp), ("intra_inv_bw", _dp),
                ("inter_alpha", _dp), ("inter_inv_bw", _dp), ("zone_alpha", _dp), ("zone_inv_bw", _dp),
                ("egress", _dp), ("intra_bw_poly", _dp), ("inter_bw_poly", _dp), ("zone_bw_poly", _dp)]


class Run(C.Structure):
    _fields_ = [("type", C.c_uint8), ("zone", C.c_uint8), ("tp_idx", C.c_uint8), ("n_stages", C.c_uint8)]


class PlanRec(C.Structure):
    _fields_ = [("P", C.c_uint8), ("mbs_idx", C.c_uint8), ("rc", C.c_uint8), ("n_runs", C.c_uint8),
                ("D", C.c_uint16), ("_pad", C.c_uint16), ("run", Run * RUN_MAX)]


class Space(C.Structure):
    _fields_ = [("n_p", C.c_uint32), ("n_mbs", C.c_uint32), ("n_tp", C.c_uint32), ("n_rc", C.c_uint32),
                ("n_d", C.c_uint32), ("seg_max", C.c_uint32), ("p_values", C.c_uint8 * NP_MAX),
                ("mbs_idx", C.c_uint8 * MBS_MAX), ("tp_idx", C.c_uint8 * TP_MAX), ("rc_values", C.c_uint8 * 2),
                ("_pad", C.c_uint8 * 6), ("d_values", C.c_uint16 * ND_MAX)]


class Objective(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("flags", C.c_uint32), ("budget_usd_per_iter", C.c_double),
                ("min_iters_per_s", C.c_double), ("budget_factor_over_cheapest", C.c_double)]


class Result(C.Structure):
    _fields_ = [("flat", C.c_uint64), ("t_iter", C.c_double), ("cost", C.c_double), ("peak_mem", C.c_uint64),
                ("score", C.c_double), ("status", C.c_uint32), ("_pad", C.c_uint32), ("plan", PlanRec)]


class Stats(C.Structure):
    _fields_ = [("n_total", C.c_uint64), ("n_invalid", C.c_uint64), ("n_oom", C.c_uint64),
                ("n_over_avail", C.c_uint64), ("n_over_constraint", C.c_uint64), ("n_feasible", C.c_uint64),
                ("budget_used", C.c_double), ("min_feasible_cost", C.c_double), ("kernel_ms", C.c_float),
                ("n_launches", C.c_uint32), ("n_pruned_tp", C.c_uint64), ("n_skipped", C.c_uint64),
                ("n_configs", C.c_uint32), ("n_configs_evaluated", C.c_uint32), ("h2d_ms", C.c_float),
                ("d2h_ms", C.c_float)]


class IssueRates(C.Structure):
    _fields_ = [("ffma_warp_inst_per_s", C.c_double), ("imad_warp_inst_per_s", C.c_double),
                ("dadd_warp_inst_per_s", C.c_double), ("ffma_ms", C.c_float), ("imad_ms", C.c_float),
                ("dadd_ms", C.c_float), ("sm_count", C.c_uint32), ("warp_inst_per_run", C.c_uint64)]


class ZoneOrder(C.Structure):
    _fields_ = [("n", C.c_uint8), ("zone", C.c_uint8 * Z_MAX), ("_pad", C.c_uint8 * 3)]


class DpResult(C.Structure):
    _fields_ = [("config", C.c_uint32), ("order", C.c_uint32), ("value", C.c_double), ("t_iter", C.c_double),
                ("cost", C.c_double), ("peak_mem", C.c_uint64), ("status", C.c_uint32), ("P", C.c_uint8),
                ("mbs_idx", C.c_uint8), ("tp_idx", C.c_uint8), ("rc", C.c_uint8), ("D", C.c_uint16),
                ("_pad", C.c_uint16), ("type", C.c_uint8 * P_MAX), ("zone", C.c_uint8 * P_MAX)]


class DpStats(C.Structure):
    _fields_ = [("n_problems", C.c_uint64), ("n_solved", C.c_uint64), ("n_over_constraint", C.c_uint64),
                ("n_states", C.c_uint64),
                ("workspace_used", C.c_uint64), ("kernel_ms", C.c_float), ("n_launches", C.c_uint32),
                ("n_batches", C.c_uint32), ("n_unfinished", C.c_uint32)]


assert C.sizeof(PlanRec) == 72 and C.sizeof(Result) == 120 and C.sizeof(Space) == 152
assert C.sizeof(ZoneOrder) == 12 and C.sizeof(DpResult) == 248 and C.sizeof(DpStats) == 56
assert C.sizeof(Objective) == 32 and C.sizeof(Stats) == 104

# numpy view of an array of plan records (same 72-byte layout)
RUN_DTYPE = np.dtype([("type", "u1"), ("zone", "u1"), ("tp_idx", "u1"), ("n_stages", "u1")])
REC_DTYPE = np.dtype([("P", "u1"), ("mbs_idx", "u1"), ("rc", "u1"), ("n_runs", "u1"), ("D", "<u2"), ("_pad", "<u2"),
                      ("run", RUN_DTYPE, (RUN_MAX,))])
assert REC_DTYPE.itemsize == 72


MIX_P_MAX, MIX_GROUPS_MAX = 96, 4
MIX_GROUP_DTYPE = np.dtype([("type", "u1"), ("tp_idx", "u1"), ("count", "<u2")])
MIX_STAGE_DTYPE = np.dtype([("zone", "u1"), ("n_groups", "u1"), ("_pad", "<u2"), ("group", MIX_GROUP_DTYPE, (MIX_GROUPS_MAX,))])


def mixed_dtype(stages: int) -> np.dtype:
    """Record of a plan with mixed replicas that has room for `stages` stages (an even number up to MIX_P_MAX, so that
    the record is a multiple of 8 bytes): the head of sailor_mixed_plan and its first stages."""
    if stages < 2 or stages > MIX_P_MAX or stages % 2:
        raise ValueError("stages per record: an even number from 2 to %d" % MIX_P_MAX)
    return np.dtype([("P", "u1"), ("mbs_idx", "u1"), ("rc", "u1"), ("_pad", "u1"), ("D", "<u2"), ("_pad2", "<u2"),
                     ("stage", MIX_STAGE_DTYPE, (stages,))])


MIX_DTYPE = mixed_dtype(MIX_P_MAX)
assert MIX_DTYPE.itemsize == 1928 and mixed_dtype(32).itemsize == 648


def pack_mixed_plans(plans, stages: int = 0) -> np.ndarray:
    """List of dicts {"P", "mbs_idx", "rc", "D", "stages": [{"zone", "groups": [(type, tp_idx, count), ...]}]}
    -> array of records with room for `stages` stages each (0: the deepest plan of the list, rounded up to even)."""
    deepest = max([p["P"] for p in plans], default=1)
    if deepest > MIX_P_MAX:
        raise ValueError("at most %d stages" % MIX_P_MAX)
    out = np.zeros(len(plans), dtype=mixed_dtype(stages or max(2, deepest + deepest % 2)))
    for j, p in enumerate(plans):
        if p["P"] > out.dtype["stage"].shape[0]:
            raise ValueError("a plan of %d stages in records of %d" % (p["P"], out.dtype["stage"].shape[0]))
        out["P"][j], out["mbs_idx"][j], out["rc"][j], out["D"][j] = p["P"], p["mbs_idx"], p["rc"], p["D"]
        for i, st in enumerate(p["stages"]):
            if len(st["groups"]) > MIX_GROUPS_MAX:
                raise ValueError("at most %d groups per stage" % MIX_GROUPS_MAX)
            out["stage"]["zone"][j, i] = st["zone"]
            out["stage"]["n_groups"][j, i] = len(st["groups"])
            for q, (g, tpi, count) in enumerate(st["groups"]):
                out["stage"]["group"]["type"][j, i, q] = g
                out["stage"]["group"]["tp_idx"][j, i, q] = tpi
                out["stage"]["group"]["count"][j, i, q] = count
    return out


class MixedGroup(C.Structure):
    _fields_ = [("type", C.c_uint8), ("tp_idx", C.c_uint8), ("count", C.c_uint16)]


class MixedStage(C.Structure):
    _fields_ = [("zone", C.c_uint8), ("n_groups", C.c_uint8), ("_pad", C.c_uint16), ("group", MixedGroup * MIX_GROUPS_MAX)]


class MixedPlan(C.Structure):
    _fields_ = [("P", C.c_uint8), ("mbs_idx", C.c_uint8), ("rc", C.c_uint8), ("_pad", C.c_uint8), ("D", C.c_uint16),
                ("_pad2", C.c_uint16), ("stage", MixedStage * MIX_P_MAX)]

    def as_dict(self) -> dict:
        return {"P": self.P, "mbs_idx": self.mbs_idx, "rc": self.rc, "D": self.D,
                "stages": [{"zone": self.stage[i].zone,
                            "groups": [(self.stage[i].group[q].type, self.stage[i].group[q].tp_idx, self.stage[i].group[q].count)
                                       for q in range(self.stage[i].n_groups)]} for i in range(self.P)]}


class MixedSpace(C.Structure):
    _fields_ = [("n_p", C.c_uint32), ("n_mbs", C.c_uint32), ("n_rc", C.c_uint32), ("n_d", C.c_uint32),
                ("seg_max", C.c_uint32), ("granularity", C.c_uint32), ("p_values", C.c_uint8 * NP_MAX),
                ("mbs_idx", C.c_uint8 * MBS_MAX), ("rc_values", C.c_uint8 * 2), ("tp_idx_of_type", C.c_uint8 * T_MAX),
                ("_pad", C.c_uint8 * 6), ("d_values", C.c_uint16 * ND_MAX)]


class MixedResult(C.Structure):
    _fields_ = [("flat", C.c_uint64), ("t_iter", C.c_double), ("cost", C.c_double), ("peak_mem", C.c_uint64),
                ("score", C.c_double), ("status", C.c_uint32), ("_pad", C.c_uint32), ("plan", MixedPlan)]


assert C.sizeof(MixedPlan) == 1928 and C.sizeof(MixedResult) == 1976 and C.sizeof(MixedSpace) == 152


class SailorError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        self.code = code
        msg = f"{where}: {sailor_strerror(code)} ({code})"
        if cuda:
            msg += f" [cudaError {cuda}]"
        super().__init__(msg)


_lib = None


def load() -> C.CDLL:
    """Load the CUDA library; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2504_17096_b200.build` "
                          "(this package has no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp = C.c_void_p
    L.sailor_create.argtypes = [C.POINTER(Model), C.POINTER(Profile), C.POINTER(Cluster), C.c_int, vp, C.POINTER(vp)]
    L.sailor_destroy.argtypes = [vp]
    L.sailor_set_availability.argtypes = [vp, _u16p]
    L.sailor_simulate.argtypes = [vp, vp, C.c_uint64, C.c_int, vp, vp, vp, vp]
    L.sailor_simulate_mixed.argtypes = [vp, vp, C.c_uint64, C.c_int, vp, vp, vp, vp]
    L.sailor_simulate_mixed_strided.argtypes = [vp, vp, C.c_uint64, C.c_uint32, C.c_int, vp, vp, vp, vp]
    L.sailor_space_size.argtypes = [vp, C.POINTER(Space), _u64p]
    L.sailor_decode.argtypes = [vp, C.POINTER(Space), C.c_uint64, C.POINTER(PlanRec)]
    L.sailor_plan.argtypes = [vp, C.POINTER(Space), C.POINTER(Objective), C.c_uint32, C.POINTER(Result), _u32p,
                              C.POINTER(Stats)]
    L.sailor_plan_range.argtypes = [vp, C.POINTER(Space), C.POINTER(Objective), C.c_uint64, C.c_uint64, C.c_uint32,
                                    C.POINTER(Result), _u32p, C.POINTER(Stats)]
    L.sailor_plan_noalloc.argtypes = L.sailor_plan.argtypes
    L.sailor_plan_dp.argtypes = [vp, C.POINTER(Space), C.POINTER(ZoneOrder), C.c_uint32, C.POINTER(Objective),
                                 C.c_uint64, C.c_uint32, C.POINTER(DpResult), _u32p, C.POINTER(DpStats)]
    L.sailor_measure_issue_rates.argtypes = [C.c_int, vp, C.c_uint32, C.POINTER(IssueRates)]
    L.sailor_mixed_space_size.argtypes = [vp, C.POINTER(MixedSpace), _u64p]
    L.sailor_mixed_decode.argtypes = [vp, C.POINTER(MixedSpace), C.c_uint64, C.POINTER(MixedPlan)]
    L.sailor_plan_mixed.argtypes = [vp, C.POINTER(MixedSpace), C.POINTER(Objective), C.c_uint32, C.POINTER(MixedResult),
                                    _u32p, C.POINTER(Stats)]
    L.sailor_strerror.argtypes = [C.c_int]
    L.sailor_strerror.restype = C.c_char_p
    L.sailor_last_cuda_error.argtypes = [vp]
    for name in EXPORTS:
        if name != "sailor_strerror":
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def sailor_strerror(code: int) -> str:
    return load().sailor_strerror(code).decode()


def _check(rc: int, where: str, ctx=None):
    if rc != OK:
        cuda = load().sailor_last_cuda_error(ctx) if (ctx and rc == E_CUDA) else 0
        raise SailorError(rc, where, cuda)


def _np(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def make_space(w) -> Space:
    """sailor_space from a workload's radix lists."""
    s = Space()
    s.n_p, s.n_mbs, s.n_tp, s.n_rc, s.n_d = len(w.p_values), len(w.mbs_idx), len(w.tp_idx), len(w.rc_values), len(w.d_values)
    s.seg_max = w.seg_max
    for name in ("p_values", "mbs_idx", "tp_idx", "rc_values", "d_values"):
        arr = getattr(s, name)
        for i, x in enumerate(getattr(w, name)):
            arr[i] = int(x)
    return s


def make_objective(w, *, flags: int = 0, kind: Optional[int] = None, budget: Optional[float] = None,
                   min_rate: Optional[float] = None, factor: Optional[float] = None) -> Objective:
    return Objective(w.objective if kind is None else kind, flags,
                     w.budget_usd_per_iter if budget is None else budget,
                     w.min_iters_per_s if min_rate is None else min_rate,
                     w.budget_factor_over_cheapest if factor is None else factor)


def pack_records(recs: dict) -> np.ndarray:
    """Dict of integer arrays (workloads.random_plans layout) -> array of 72-byte plan records."""
    n = len(recs["P"])
    out = np.zeros(n, dtype=REC_DTYPE)
    for k in ("P", "mbs_idx", "rc", "n_runs", "D"):
        out[k] = recs[k]
    for k in ("type", "zone", "tp_idx", "n_stages"):
        out["run"][k] = recs[k]
    return out


def sailor_create(w, device: int = 0, stream: int = 0) -> C.c_void_p:
    """Context for a workload's model, profile and cluster tables (host arrays are copied)."""
    m = Model(w.n_blocks, w.has_embed, w.has_head, w.heads, w.gbs, w.mul_factor, w.dtype_size, w.grad_dtype_size, 0)
    keep = []

    def ptr(a, dtype, ptype):
        a = _np(a, dtype)
        keep.append(a)
        return a.ctypes.data_as(ptype)

    p = Profile()
    p.n_types, p.n_tp, p.n_mbs = w.n_types, len(w.tp_values), len(w.mbs_values)
    for i, x in enumerate(w.tp_values):
        p.tp_values[i] = x
    for i, x in enumerate(w.mbs_values):
        p.mbs_values[i] = x
    p.fwd, p.bwd, p.upd = ptr(w.fwd, np.float64, _dp), ptr(w.bwd, np.float64, _dp), ptr(w.upd, np.float64, _dp)
    p.params = ptr(w.params, np.uint64, _u64p)
    p.act_saved, p.act_ckpt = ptr(w.act_saved, np.uint64, _u64p), ptr(w.act_ckpt, np.uint64, _u64p)
    p.act_work, p.p2p_bytes = ptr(w.act_work, np.uint64, _u64p), ptr(w.p2p_bytes, np.uint64, _u64p)
    c = Cluster()
    c.n_types, c.n_zones = w.n_types, w.n_zones
    c.capacity, c.reserved = ptr(w.capacity, np.uint64, _u64p), ptr(w.reserved, np.uint64, _u64p)
    c.gpus_per_node = ptr(w.gpus_per_node, np.uint32, _u32p)
    for name in ("price_per_hour", "intra_alpha", "intra_inv_bw", "inter_alpha", "inter_inv_bw", "zone_alpha",
                 "zone_inv_bw", "egress"):
        setattr(c, name, ptr(getattr(w, name), np.float64, _dp))
    for name in ("intra_bw_poly", "inter_bw_poly", "zone_bw_poly"):       # optional: NULL when absent
        if getattr(w, name, None) is not None:
            setattr(c, name, ptr(getattr(w, name), np.float64, _dp))
    ctx = C.c_void_p()
    _check(load().sailor_create(C.byref(m), C.byref(p), C.byref(c), device, C.c_void_p(stream), C.byref(ctx)),
           "sailor_create")
    return ctx


def sailor_destroy(ctx) -> None:
    _check(load().sailor_destroy(ctx), "sailor_destroy")


def sailor_set_availability(ctx, avail) -> None:
    a = _np(avail, np.uint16)
    _check(load().sailor_set_availability(ctx, a.ctypes.data_as(_u16p)), "sailor_set_availability", ctx)


def sailor_simulate(ctx, plans: np.ndarray):
    """Host path: records (REC_DTYPE array) in, (t_iter, peak_mem, cost, status) numpy arrays out."""
    plans = np.ascontiguousarray(plans, dtype=REC_DTYPE)
    n = plans.size
    t, c = np.empty(n, np.float64), np.empty(n, np.float64)
    m, s = np.empty(n, np.uint64), np.empty(n, np.uint32)
    _check(load().sailor_simulate(ctx, plans.ctypes.data, n, 0, t.ctypes.data, m.ctypes.data, c.ctypes.data,
                                  s.ctypes.data), "sailor_simulate", ctx)
    return t, m, c, s


def sailor_simulate_host(ctx, plans_ptr: int, n: int, t_iter_ptr: int, peak_mem_ptr: int, cost_ptr: int,
                         status_ptr: int) -> None:
    """Host path on raw host pointers (e.g. pinned buffers): copies in, simulates, copies out, returns when done."""
    _check(load().sailor_simulate(ctx, plans_ptr, n, 0, t_iter_ptr or None, peak_mem_ptr or None, cost_ptr or None,
                                  status_ptr or None), "sailor_simulate", ctx)


def sailor_simulate_device(ctx, plans_ptr: int, n: int, t_iter_ptr: int, peak_mem_ptr: int, cost_ptr: int,
                           status_ptr: int) -> None:
    """Device path: raw device pointers (e.g. torch tensors' data_ptr()); only enqueues work."""
    _check(load().sailor_simulate(ctx, plans_ptr, n, 1, t_iter_ptr or None, peak_mem_ptr or None, cost_ptr or None,
                                  status_ptr or None), "sailor_simulate", ctx)


def sailor_simulate_mixed(ctx, plans: np.ndarray):
    """Plans with mixed replicas (an array of a mixed_dtype, see pack_mixed_plans) in, (t_iter, peak_mem, cost, status)
    out.  Records shorter than sailor_mixed_plan go through sailor_simulate_mixed_strided."""
    plans = np.ascontiguousarray(plans)
    if "stage" not in (plans.dtype.names or ()) or plans.dtype != mixed_dtype(plans.dtype["stage"].shape[0]):
        raise TypeError("an array made by pack_mixed_plans is wanted")
    n = plans.size
    t, c = np.empty(n, np.float64), np.empty(n, np.float64)
    m, s = np.empty(n, np.uint64), np.empty(n, np.uint32)
    if plans.dtype.itemsize == C.sizeof(MixedPlan):
        rc = load().sailor_simulate_mixed(ctx, plans.ctypes.data, n, 0, t.ctypes.data, m.ctypes.data, c.ctypes.data, s.ctypes.data)
    else:
        rc = load().sailor_simulate_mixed_strided(ctx, plans.ctypes.data, n, plans.dtype.itemsize, 0, t.ctypes.data,
                                                  m.ctypes.data, c.ctypes.data, s.ctypes.data)
    _check(rc, "sailor_simulate_mixed", ctx)
    return t, m, c, s


def sailor_simulate_mixed_device(ctx, plans_ptr: int, n: int, t_iter_ptr: int, peak_mem_ptr: int, cost_ptr: int,
                                 status_ptr: int, record_bytes: int = 0) -> None:
    """Device path of sailor_simulate_mixed (record_bytes 0: whole sailor_mixed_plan records) and of
    sailor_simulate_mixed_strided: raw device pointers; only enqueues work."""
    _check(load().sailor_simulate_mixed_strided(ctx, plans_ptr, n, record_bytes or C.sizeof(MixedPlan), 1, t_iter_ptr or None,
                                                peak_mem_ptr or None, cost_ptr or None, status_ptr or None),
           "sailor_simulate_mixed", ctx)


def sailor_space_size(ctx, space: Space) -> int:
    n = C.c_uint64()
    _check(load().sailor_space_size(ctx, C.byref(space), C.byref(n)), "sailor_space_size")
    return int(n.value)


def sailor_decode(ctx, space: Space, flat: int) -> PlanRec:
    r = PlanRec()
    _check(load().sailor_decode(ctx, C.byref(space), flat, C.byref(r)), "sailor_decode")
    return r


def sailor_plan_range(ctx, space: Space, obj: Objective, lo: int, hi: int, k: int):
    res = (Result * k)()
    n = C.c_uint32()
    st = Stats()
    _check(load().sailor_plan_range(ctx, C.byref(space), C.byref(obj), lo, hi, k, res, C.byref(n), C.byref(st)),
           "sailor_plan_range", ctx)
    return list(res[: n.value]), st


def sailor_plan(ctx, space: Space, obj: Objective, k: int):
    res = (Result * k)()
    n = C.c_uint32()
    st = Stats()
    _check(load().sailor_plan(ctx, C.byref(space), C.byref(obj), k, res, C.byref(n), C.byref(st)), "sailor_plan", ctx)
    return list(res[: n.value]), st


def sailor_plan_noalloc(ctx, space: Space, obj: Objective, k: int):
    """The search of sailor_plan for callers that must not allocate device memory: all working
    memory comes from a fixed array inside the library (spaces of at most 4096 configurations;
    calls on one GPU must not overlap).  Same return values as sailor_plan."""
    res = (Result * k)()
    n = C.c_uint32()
    st = Stats()
    _check(load().sailor_plan_noalloc(ctx, C.byref(space), C.byref(obj), k, res, C.byref(n), C.byref(st)),
           "sailor_plan_noalloc", ctx)
    return list(res[: n.value]), st


def all_zone_orders(n_zones: int, max_len: Optional[int] = None):
    """Every ordered selection of 1 .. max_len distinct zones (the region combinations a planner would loop over):
    n_zones = 3 gives 15 orders, 4 gives 64, 5 gives 325."""
    import itertools
    max_len = n_zones if max_len is None else min(max_len, n_zones)
    return [list(p) for n in range(1, max_len + 1) for p in itertools.permutations(range(n_zones), n)]


def make_mixed_space(w, granularity: int, tp_idx_of_type, *, p_values=None, mbs_idx=None, rc_values=None,
                     d_values=None, seg_max=None) -> MixedSpace:
    """sailor_mixed_space from a workload's radix lists (or the given ones)."""
    s = MixedSpace()
    lists = {"p_values": w.p_values if p_values is None else p_values, "mbs_idx": w.mbs_idx if mbs_idx is None else mbs_idx,
             "rc_values": w.rc_values if rc_values is None else rc_values, "d_values": w.d_values if d_values is None else d_values,
             "tp_idx_of_type": tp_idx_of_type}
    for name, values in lists.items():
        arr = getattr(s, name)
        for i, x in enumerate(values):
            arr[i] = int(x)
    s.n_p, s.n_mbs, s.n_rc, s.n_d = (len(lists[k]) for k in ("p_values", "mbs_idx", "rc_values", "d_values"))
    s.seg_max = w.seg_max if seg_max is None else seg_max
    s.granularity = granularity
    return s


def sailor_mixed_space_size(ctx, space: MixedSpace) -> int:
    n = C.c_uint64()
    _check(load().sailor_mixed_space_size(ctx, C.byref(space), C.byref(n)), "sailor_mixed_space_size")
    return int(n.value)


def sailor_mixed_decode(ctx, space: MixedSpace, flat: int) -> MixedPlan:
    r = MixedPlan()
    _check(load().sailor_mixed_decode(ctx, C.byref(space), flat, C.byref(r)), "sailor_mixed_decode")
    return r


def sailor_plan_mixed(ctx, space: MixedSpace, obj: Objective, k: int):
    """Search over plans whose stages mix GPU types among their replicas: the k best and the statistics."""
    res = (MixedResult * k)()
    n = C.c_uint32()
    st = Stats()
    _check(load().sailor_plan_mixed(ctx, C.byref(space), C.byref(obj), k, res, C.byref(n), C.byref(st)),
           "sailor_plan_mixed", ctx)
    return list(res[: n.value]), st


def sailor_measure_issue_rates(device: int = 0, stream: int = 0, repeats: int = 5) -> IssueRates:
    """Sustained warp-instructions per second of an FP32 multiply-add, an integer multiply-add and an FP64 add
    stream on the device (CUDA events, best of `repeats`)."""
    r = IssueRates()
    _check(load().sailor_measure_issue_rates(device, C.c_void_p(stream), repeats, C.byref(r)), "sailor_measure_issue_rates")
    return r


dp_default_flags = 0      # SAILOR_DP_FLAG_* that sailor_plan_dp passes when the caller gives no objective


def sailor_plan_dp(ctx, space: Space, zone_orders, k: int, workspace_bytes: int = 0, *, budget: float = 0.0,
                   min_rate: float = 0.0, obj: Optional[Objective] = None, budget_loop: bool = False):
    """Per-stage GPU types by dynamic programming for every configuration of the space and every zone
    order (a list of zone lists): the k best plans by the recursion's value among those within the
    budget / minimum throughput, and the statistics."""
    if obj is None:
        obj = Objective(OBJ_MAX_THROUGHPUT, DP_FLAG_BUDGET_LOOP if budget_loop else dp_default_flags, budget, min_rate, 0.0)
    orders = (ZoneOrder * len(zone_orders))()
    for j, zl in enumerate(zone_orders):
        if len(zl) > Z_MAX:
            raise ValueError("a zone order holds at most %d zones" % Z_MAX)
        orders[j].n = len(zl)
        for q, z in enumerate(zl):
            orders[j].zone[q] = int(z)
    res = (DpResult * k)()
    n = C.c_uint32()
    st = DpStats()
    _check(load().sailor_plan_dp(ctx, C.byref(space), orders, len(zone_orders), C.byref(obj), workspace_bytes, k, res,
                                 C.byref(n), C.byref(st)), "sailor_plan_dp", ctx)
    return list(res[: n.value]), st


def stats_dict(st: Stats) -> dict:
    return {f: getattr(st, f) for f, _ in Stats._fields_}
