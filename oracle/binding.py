"""ctypes binding of the CPU oracle — TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It compiles ``sailor_oracle.c`` with gcc on first use and marshals a workload (plain numbers
and numpy arrays) into the oracle's own structures.  It imports nothing from the CUDA
package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sailor_oracle.c")
_HDR = os.path.join(_HERE, "sailor_oracle.h")
_LIB = os.path.join(_HERE, "liboracle.so")

STAGES_MAX = 128
ST_INVALID, ST_OVER_AVAIL, ST_OOM = 1, 2, 4


def build(force: bool = False) -> str:
    """Compile the oracle (contraction off, no fast-math) if the library is missing or stale."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math",
                               "-Wall", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_dp = C.POINTER(C.c_double)
_u64p = C.POINTER(C.c_uint64)
_u32p = C.POINTER(C.c_uint32)
_u16p = C.POINTER(C.c_uint16)


class OrcInputs(C.Structure):
    _fields_ = [
        ("n_blocks", C.c_uint32), ("has_embed", C.c_uint32), ("has_head", C.c_uint32), ("heads", C.c_uint32),
        ("gbs", C.c_uint64),
        ("mul_factor", C.c_uint32), ("dtype_size", C.c_uint32), ("grad_dtype_size", C.c_uint32),
        ("n_types", C.c_uint32), ("n_zones", C.c_uint32), ("n_tp", C.c_uint32), ("n_mbs", C.c_uint32),
        ("tp_values", _u32p), ("mbs_values", _u32p),
        ("fwd", _dp), ("bwd", _dp), ("upd", _dp),
        ("params", _u64p), ("act_saved", _u64p), ("act_ckpt", _u64p), ("act_work", _u64p), ("p2p_bytes", _u64p),
        ("capacity", _u64p), ("reserved", _u64p), ("gpus_per_node", _u32p),
        ("price_per_hour", _dp), ("intra_alpha", _dp), ("intra_inv_bw", _dp), ("inter_alpha", _dp),
        ("inter_inv_bw", _dp), ("zone_alpha", _dp), ("zone_inv_bw", _dp), ("egress", _dp),
        ("intra_bw_poly", _dp), ("inter_bw_poly", _dp), ("zone_bw_poly", _dp),
        ("avail", _u16p),
    ]


class OrcPlan(C.Structure):
    _fields_ = [("P", C.c_uint32), ("mbs_idx", C.c_uint32), ("rc", C.c_uint32), ("D", C.c_uint32),
                ("type", C.c_uint32 * STAGES_MAX), ("zone", C.c_uint32 * STAGES_MAX),
                ("tp_idx", C.c_uint32 * STAGES_MAX)]


class OrcOut(C.Structure):
    _fields_ = [("status", C.c_uint32), ("_pad", C.c_uint32), ("t_iter", C.c_double), ("cost", C.c_double),
                ("peak_mem", C.c_uint64), ("t_pp", C.c_double), ("t_sync", C.c_double),
                ("t_update", C.c_double), ("rate_per_s", C.c_double), ("c_comm", C.c_double),
                ("n_b", C.c_uint64), ("stage_mem", C.c_uint64 * STAGES_MAX),
                ("stage_t", C.c_double * STAGES_MAX), ("stage_c", C.c_double * STAGES_MAX),
                ("stage_sync", C.c_double * STAGES_MAX)]


class OrcSpace(C.Structure):
    _fields_ = [("n_p", C.c_uint32), ("n_mbs", C.c_uint32), ("n_tp", C.c_uint32), ("n_rc", C.c_uint32),
                ("n_d", C.c_uint32), ("seg_max", C.c_uint32),
                ("p_values", _u32p), ("mbs_idx", _u32p), ("tp_idx", _u32p), ("rc_values", _u32p),
                ("d_values", _u32p)]


class OrcObjective(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("_pad", C.c_uint32), ("budget", C.c_double), ("min_rate", C.c_double)]


class OrcHit(C.Structure):
    _fields_ = [("flat", C.c_uint64), ("score", C.c_double), ("t_iter", C.c_double), ("cost", C.c_double),
                ("peak_mem", C.c_uint64)]


class OrcCounts(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("n_total", "n_invalid", "n_oom", "n_over_avail",
                                          "n_over_constraint", "n_feasible")] + [("min_cost", C.c_double)]


class OrcPrunedCounts(C.Structure):
    _fields_ = [("looked_at", OrcCounts), ("n_pruned_tp", C.c_uint64), ("n_skipped", C.c_uint64),
                ("n_configs", C.c_uint64), ("n_configs_evaluated", C.c_uint64)]


PRUNE_D_ORDER, PRUNE_MIN_TP = 1, 2


class OrcDpProblem(C.Structure):
    _fields_ = [("P", C.c_uint32), ("mbs_idx", C.c_uint32), ("tp_idx", C.c_uint32), ("rc", C.c_uint32),
                ("D", C.c_uint32), ("n_zones_used", C.c_uint32), ("zone_list", C.c_uint32 * 16)]


class OrcDpResult(C.Structure):
    _fields_ = [("found", C.c_int32), ("_pad", C.c_uint32), ("value", C.c_double), ("n_states", C.c_uint64),
                ("plan", OrcPlan)]


class OrcDpBudgetResult(C.Structure):
    _fields_ = [("found", C.c_int32), ("_pad", C.c_uint32), ("value", C.c_double), ("charged_cost", C.c_double),
                ("n_states", C.c_uint64), ("plan", OrcPlan)]


GROUPS_MAX = 4


class OrcReplicaGroup(C.Structure):
    _fields_ = [("type", C.c_uint32), ("tp_idx", C.c_uint32), ("count", C.c_uint32)]


class OrcMixedStage(C.Structure):
    _fields_ = [("zone", C.c_uint32), ("n_groups", C.c_uint32), ("group", OrcReplicaGroup * GROUPS_MAX)]


class OrcMixedPlan(C.Structure):
    _fields_ = [("P", C.c_uint32), ("mbs_idx", C.c_uint32), ("rc", C.c_uint32), ("D", C.c_uint32),
                ("stage", OrcMixedStage * STAGES_MAX)]


class OrcMixedSpace(C.Structure):
    _fields_ = [("n_p", C.c_uint32), ("n_mbs", C.c_uint32), ("n_rc", C.c_uint32), ("n_d", C.c_uint32),
                ("seg_max", C.c_uint32), ("granularity", C.c_uint32), ("p_values", _u32p), ("mbs_idx", _u32p),
                ("rc_values", _u32p), ("d_values", _u32p), ("tp_idx_of_type", _u32p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_simulate.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcPlan), C.POINTER(OrcOut)]
        L.orc_simulate.restype = None
        L.orc_space_size.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcSpace)]
        L.orc_space_size.restype = C.c_uint64
        L.orc_decode.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcSpace), C.c_uint64, C.POINTER(OrcPlan)]
        L.orc_decode.restype = C.c_int
        L.orc_search.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcSpace), C.POINTER(OrcObjective),
                                 C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32, C.POINTER(OrcHit),
                                 C.POINTER(OrcCounts)]
        L.orc_search.restype = C.c_uint32
        L.orc_simulate_flat.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcSpace), _u64p, C.c_uint64,
                                        _u32p, _dp, _dp, _u64p]
        L.orc_simulate_flat.restype = None
        L.orc_simulate_batch.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcPlan), C.c_uint64,
                                         _u32p, _dp, _dp, _u64p]
        L.orc_simulate_batch.restype = None
        L.orc_search_pruned.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcSpace), C.POINTER(OrcObjective),
                                        C.c_uint32, C.c_uint32, C.POINTER(OrcHit), C.POINTER(OrcPrunedCounts)]
        L.orc_search_pruned.restype = C.c_int32
        L.orc_solve_dp.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcDpProblem), C.c_int, C.POINTER(OrcDpResult)]
        L.orc_solve_dp.restype = C.c_int
        L.orc_solve_dp_budget.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcDpProblem), C.c_double,
                                          C.POINTER(OrcDpBudgetResult)]
        L.orc_solve_dp_budget.restype = C.c_int
        L.orc_simulate_mixed.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcMixedPlan), C.POINTER(OrcOut)]
        L.orc_simulate_mixed.restype = None
        L.orc_simulate_mixed_batch.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcMixedPlan), C.c_uint64,
                                               _u32p, _dp, _dp, _u64p]
        L.orc_simulate_mixed_batch.restype = None
        L.orc_mixed_n_comb.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcMixedSpace), C.c_uint32]
        L.orc_mixed_n_comb.restype = C.c_uint64
        L.orc_mixed_comb.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcMixedSpace), C.c_uint32, C.c_uint64, _u32p]
        L.orc_mixed_comb.restype = C.c_int
        L.orc_mixed_space_size.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcMixedSpace)]
        L.orc_mixed_space_size.restype = C.c_uint64
        L.orc_mixed_decode.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcMixedSpace), C.c_uint64, C.POINTER(OrcMixedPlan)]
        L.orc_mixed_decode.restype = C.c_int
        L.orc_search_mixed.argtypes = [C.POINTER(OrcInputs), C.POINTER(OrcMixedSpace), C.POINTER(OrcObjective),
                                       C.c_uint64, C.c_uint64, C.c_uint32, C.POINTER(OrcHit), C.POINTER(OrcCounts)]
        L.orc_search_mixed.restype = C.c_uint32
        _lib = L
    return _lib


def _arr(a, dtype, ptr_type):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, a.ctypes.data_as(ptr_type)


class Oracle:
    """The oracle bound to one workload's tables (kept alive here)."""

    def __init__(self, w, avail: Optional[np.ndarray] = None):
        self._keep = []
        self.w = w
        i = OrcInputs()
        for name in ("n_blocks", "has_embed", "has_head", "heads", "gbs", "mul_factor", "dtype_size",
                     "grad_dtype_size", "n_types", "n_zones"):
            setattr(i, name, int(getattr(w, name)))
        if w.n_blocks > 1024:
            raise ValueError("oracle supports at most 1024 blocks")
        i.n_tp, i.n_mbs = len(w.tp_values), len(w.mbs_values)

        def put(name, value, dtype, ptr):
            a, p = _arr(value, dtype, ptr)
            self._keep.append(a)
            setattr(i, name, p)
            return a

        put("tp_values", w.tp_values, np.uint32, _u32p)
        put("mbs_values", w.mbs_values, np.uint32, _u32p)
        for name in ("fwd", "bwd", "upd", "price_per_hour", "intra_alpha", "intra_inv_bw", "inter_alpha",
                     "inter_inv_bw", "zone_alpha", "zone_inv_bw", "egress"):
            put(name, getattr(w, name), np.float64, _dp)
        for name in ("params", "act_saved", "act_ckpt", "act_work", "p2p_bytes", "capacity", "reserved"):
            put(name, getattr(w, name), np.uint64, _u64p)
        put("gpus_per_node", w.gpus_per_node, np.uint32, _u32p)
        for name in ("intra_bw_poly", "inter_bw_poly", "zone_bw_poly"):
            if getattr(w, name, None) is not None:
                put(name, getattr(w, name), np.float64, _dp)
        self._avail = put("avail", np.array(w.avail if avail is None else avail, dtype=np.uint16, copy=True),
                          np.uint16, _u16p)
        self.inputs = i

        s = OrcSpace()
        s.n_p, s.n_mbs, s.n_tp = len(w.p_values), len(w.mbs_idx), len(w.tp_idx)
        s.n_rc, s.n_d, s.seg_max = len(w.rc_values), len(w.d_values), w.seg_max
        for name in ("p_values", "mbs_idx", "tp_idx", "rc_values", "d_values"):
            a, p = _arr(getattr(w, name), np.uint32, _u32p)
            self._keep.append(a)
            setattr(s, name, p)
        self.space = s

    def set_availability(self, avail) -> None:
        self._avail[...] = np.asarray(avail, dtype=np.uint16).reshape(self._avail.shape)

    # -- single plans -------------------------------------------------------------------
    @staticmethod
    def make_plan(P: int, mbs_idx: int, rc: int, D: int, types: Sequence[int], zones: Sequence[int],
                  tp_idx: Sequence[int]) -> OrcPlan:
        pl = OrcPlan()
        pl.P, pl.mbs_idx, pl.rc, pl.D = P, mbs_idx, rc, D
        for j in range(P):
            pl.type[j], pl.zone[j], pl.tp_idx[j] = int(types[j]), int(zones[j]), int(tp_idx[j])
        return pl

    def simulate(self, plan: OrcPlan) -> OrcOut:
        out = OrcOut()
        lib().orc_simulate(C.byref(self.inputs), C.byref(plan), C.byref(out))
        return out

    # -- plans whose stages mix GPU types among their replicas ---------------------------
    @staticmethod
    def make_mixed_plan(plan: dict) -> OrcMixedPlan:
        """plan = {"P", "mbs_idx", "rc", "D", "stages": [{"zone", "groups": [(type, tp_idx, count), ...]}, ...]}"""
        pl = OrcMixedPlan()
        pl.P, pl.mbs_idx, pl.rc, pl.D = plan["P"], plan["mbs_idx"], plan["rc"], plan["D"]
        for i, st in enumerate(plan["stages"]):
            if len(st["groups"]) > GROUPS_MAX:
                raise ValueError("too many groups in a stage")
            pl.stage[i].zone = int(st["zone"])
            pl.stage[i].n_groups = len(st["groups"])
            for q, (g, tpi, count) in enumerate(st["groups"]):
                pl.stage[i].group[q].type, pl.stage[i].group[q].tp_idx, pl.stage[i].group[q].count = int(g), int(tpi), int(count)
        return pl

    def simulate_mixed(self, plan: dict) -> OrcOut:
        out = OrcOut()
        pl = self.make_mixed_plan(plan)
        lib().orc_simulate_mixed(C.byref(self.inputs), C.byref(pl), C.byref(out))
        return out

    def simulate_mixed_batch(self, plans):
        n = len(plans)
        arr = (OrcMixedPlan * n)()
        for j, p in enumerate(plans):
            arr[j] = self.make_mixed_plan(p)
        st = np.zeros(n, np.uint32); t = np.zeros(n); c = np.zeros(n); m = np.zeros(n, np.uint64)
        lib().orc_simulate_mixed_batch(C.byref(self.inputs), arr, n, st.ctypes.data_as(_u32p), t.ctypes.data_as(_dp),
                                       c.ctypes.data_as(_dp), m.ctypes.data_as(_u64p))
        return st, t, c, m

    def space_size(self) -> int:
        return int(lib().orc_space_size(C.byref(self.inputs), C.byref(self.space)))

    def decode(self, flat: int) -> OrcPlan:
        pl = OrcPlan()
        if lib().orc_decode(C.byref(self.inputs), C.byref(self.space), flat, C.byref(pl)) != 0:
            raise IndexError(flat)
        return pl

    # -- batches ------------------------------------------------------------------------
    def simulate_flat(self, flat) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
        flat = np.ascontiguousarray(flat, dtype=np.uint64)
        n = flat.size
        st = np.zeros(n, np.uint32); t = np.zeros(n); c = np.zeros(n); m = np.zeros(n, np.uint64)
        lib().orc_simulate_flat(C.byref(self.inputs), C.byref(self.space), flat.ctypes.data_as(_u64p), n,
                                st.ctypes.data_as(_u32p), t.ctypes.data_as(_dp), c.ctypes.data_as(_dp),
                                m.ctypes.data_as(_u64p))
        return st, t, c, m

    def simulate_records(self, recs: dict):
        """Simulate run-length encoded records (the dict layout of workloads.random_plans)."""
        n = len(recs["P"])
        plans = (OrcPlan * n)()
        for j in range(n):
            pl = plans[j]
            pl.P, pl.mbs_idx, pl.rc, pl.D = (int(recs["P"][j]), int(recs["mbs_idx"][j]), int(recs["rc"][j]),
                                             int(recs["D"][j]))
            i = 0
            for r in range(int(recs["n_runs"][j])):
                for _ in range(int(recs["n_stages"][j, r])):
                    pl.type[i] = int(recs["type"][j, r])
                    pl.zone[i] = int(recs["zone"][j, r])
                    pl.tp_idx[i] = int(recs["tp_idx"][j, r])
                    i += 1
        st = np.zeros(n, np.uint32); t = np.zeros(n); c = np.zeros(n); m = np.zeros(n, np.uint64)
        lib().orc_simulate_batch(C.byref(self.inputs), plans, n, st.ctypes.data_as(_u32p),
                                 t.ctypes.data_as(_dp), c.ctypes.data_as(_dp), m.ctypes.data_as(_u64p))
        return st, t, c, m

    # -- search -------------------------------------------------------------------------
    def search(self, kind: int, k: int, *, budget: float = 0.0, min_rate: float = 0.0, lo: int = 0,
               hi: Optional[int] = None, stride: int = 1):
        """One exhaustive pass over [lo, hi): returns (hits as list of dicts, counts dict)."""
        hi = self.space_size() if hi is None else hi
        obj = OrcObjective(kind, 0, budget, min_rate)
        hits = (OrcHit * max(k, 1))()
        cnt = OrcCounts()
        n = lib().orc_search(C.byref(self.inputs), C.byref(self.space), C.byref(obj), lo, hi, stride, k,
                             hits, C.byref(cnt))
        out = [dict(flat=int(h.flat), score=h.score, t_iter=h.t_iter, cost=h.cost, peak_mem=int(h.peak_mem))
               for h in hits[:n]]
        return out, {f: (getattr(cnt, f) if f == "min_cost" else int(getattr(cnt, f))) for f, _ in OrcCounts._fields_}

    def search_pruned(self, kind: int, k: int, modes: int, *, budget: float = 0.0, min_rate: float = 0.0):
        """Whole-space search with the planner's pruning heuristics as modes (PRUNE_D_ORDER: H3/H4,
        PRUNE_MIN_TP: H2 extended): returns (hits, counts dict)."""
        obj = OrcObjective(kind, 0, budget, min_rate)
        hits = (OrcHit * max(k, 1))()
        cnt = OrcPrunedCounts()
        n = lib().orc_search_pruned(C.byref(self.inputs), C.byref(self.space), C.byref(obj), modes, k, hits,
                                    C.byref(cnt))
        if n < 0:
            raise ValueError("the pruning mode is not defined for this objective")
        out = [dict(flat=int(h.flat), score=h.score, t_iter=h.t_iter, cost=h.cost, peak_mem=int(h.peak_mem))
               for h in hits[:n]]
        counts = {f: (getattr(cnt.looked_at, f) if f == "min_cost" else int(getattr(cnt.looked_at, f)))
                  for f, _ in OrcCounts._fields_}
        for f in ("n_pruned_tp", "n_skipped", "n_configs", "n_configs_evaluated"):
            counts[f] = int(getattr(cnt, f))
        return out, counts

    def solve_dp(self, P: int, mbs_idx: int, tp_idx: int, rc: int, D: int, zone_list: Sequence[int], *,
                 use_memo: bool = True) -> Optional[dict]:
        """Per-stage GPU types by the dynamic-programming recursion (Sec. 4.2.2) for one configuration and
        one zone order; None when no plan fits.  Returns value, types, zones, the written-out plan and the
        number of states solved."""
        pb = OrcDpProblem()
        pb.P, pb.mbs_idx, pb.tp_idx, pb.rc, pb.D, pb.n_zones_used = P, mbs_idx, tp_idx, rc, D, len(zone_list)
        for j, z in enumerate(zone_list):
            pb.zone_list[j] = int(z)
        out = OrcDpResult()
        if lib().orc_solve_dp(C.byref(self.inputs), C.byref(pb), 1 if use_memo else 0, C.byref(out)) != 0:
            raise ValueError("problem beyond the oracle's limits")
        if not out.found:
            return None
        plan = OrcPlan.from_buffer_copy(out.plan)
        return {"value": out.value, "types": list(plan.type[:P]), "zones": list(plan.zone[:P]), "plan": plan,
                "n_states": int(out.n_states)}

    def solve_dp_budget(self, P: int, mbs_idx: int, tp_idx: int, rc: int, D: int, zone_list: Sequence[int],
                        limit: float) -> Optional[dict]:
        """The recursion under a cost limit (Sec. 4.2.3: stages charged by the assumed straggler, re-solved when
        the straggler turns out different); None when no plan is within the limit."""
        pb = OrcDpProblem()
        pb.P, pb.mbs_idx, pb.tp_idx, pb.rc, pb.D, pb.n_zones_used = P, mbs_idx, tp_idx, rc, D, len(zone_list)
        for j, z in enumerate(zone_list):
            pb.zone_list[j] = int(z)
        out = OrcDpBudgetResult()
        if lib().orc_solve_dp_budget(C.byref(self.inputs), C.byref(pb), float(limit), C.byref(out)) != 0:
            raise ValueError("problem beyond the oracle's limits")
        if not out.found:
            return None
        plan = OrcPlan.from_buffer_copy(out.plan)
        return {"value": out.value, "charged_cost": out.charged_cost, "types": list(plan.type[:P]),
                "zones": list(plan.zone[:P]), "plan": plan, "n_states": int(out.n_states)}

    # -- search over plans with mixed replicas ----------------------------------------------
    def mixed_space(self, granularity: int, tp_idx_of_type: Sequence[int], *, p_values=None, mbs_idx=None,
                    rc_values=None, d_values=None, seg_max=None) -> OrcMixedSpace:
        """The workload's radix lists (or the given ones) as a space of plans with mixed replicas."""
        w = self.w
        s = OrcMixedSpace()
        lists = {"p_values": w.p_values if p_values is None else p_values,
                 "mbs_idx": w.mbs_idx if mbs_idx is None else mbs_idx,
                 "rc_values": w.rc_values if rc_values is None else rc_values,
                 "d_values": w.d_values if d_values is None else d_values,
                 "tp_idx_of_type": tp_idx_of_type}
        for name, value in lists.items():
            a, p = _arr(value, np.uint32, _u32p)
            self._keep.append(a)
            setattr(s, name, p)
        s.n_p, s.n_mbs, s.n_rc, s.n_d = (len(lists[k]) for k in ("p_values", "mbs_idx", "rc_values", "d_values"))
        s.seg_max = w.seg_max if seg_max is None else seg_max
        s.granularity = granularity
        return s

    def mixed_n_comb(self, space: OrcMixedSpace, D: int) -> int:
        return int(lib().orc_mixed_n_comb(C.byref(self.inputs), C.byref(space), D))

    def mixed_comb(self, space: OrcMixedSpace, D: int, c: int):
        u = (C.c_uint32 * 8)()
        if lib().orc_mixed_comb(C.byref(self.inputs), C.byref(space), D, c, u) != 0:
            raise IndexError(c)
        return list(u[: self.w.n_types])

    def mixed_space_size(self, space: OrcMixedSpace) -> int:
        return int(lib().orc_mixed_space_size(C.byref(self.inputs), C.byref(space)))

    def mixed_decode(self, space: OrcMixedSpace, flat: int) -> dict:
        pl = OrcMixedPlan()
        if lib().orc_mixed_decode(C.byref(self.inputs), C.byref(space), flat, C.byref(pl)) != 0:
            raise IndexError(flat)
        return {"P": pl.P, "mbs_idx": pl.mbs_idx, "rc": pl.rc, "D": pl.D,
                "stages": [{"zone": pl.stage[i].zone,
                            "groups": [(pl.stage[i].group[q].type, pl.stage[i].group[q].tp_idx, pl.stage[i].group[q].count)
                                       for q in range(pl.stage[i].n_groups)]} for i in range(pl.P)]}

    def search_mixed(self, space: OrcMixedSpace, kind: int, k: int, *, budget: float = 0.0, min_rate: float = 0.0,
                     lo: int = 0, hi: Optional[int] = None):
        hi = self.mixed_space_size(space) if hi is None else hi
        obj = OrcObjective(kind, 0, budget, min_rate)
        hits = (OrcHit * max(k, 1))()
        cnt = OrcCounts()
        n = lib().orc_search_mixed(C.byref(self.inputs), C.byref(space), C.byref(obj), lo, hi, k, hits, C.byref(cnt))
        out = [dict(flat=int(h.flat), score=h.score, t_iter=h.t_iter, cost=h.cost, peak_mem=int(h.peak_mem))
               for h in hits[:n]]
        return out, {f: (getattr(cnt, f) if f == "min_cost" else int(getattr(cnt, f))) for f, _ in OrcCounts._fields_}

    def plan(self, k: int, *, lo: int = 0, hi: Optional[int] = None):
        """The workload's own objective, with the cheapest-feasible budget rule when it has one:
        pass 1 minimises cost without a budget, pass 2 runs the objective under
        budget = factor x that cost (Sec. 5.2.4, scenario 2 shape)."""
        w = self.w
        budget = w.budget_usd_per_iter
        if w.budget_factor_over_cheapest > 0.0:
            cheapest, _ = self.search(1, 1, lo=lo, hi=hi)
            if not cheapest:
                return [], {"n_feasible": 0}, 0.0
            budget = w.budget_factor_over_cheapest * cheapest[0]["cost"]
        hits, counts = self.search(w.objective, k, budget=budget, min_rate=w.min_iters_per_s, lo=lo, hi=hi)
        return hits, counts, budget


def merge_hits(lists: List[list], k: int) -> list:
    """Merge per-range top-k lists by (score, flat)."""
    allh = [h for l in lists for h in l]
    allh.sort(key=lambda h: (h["score"], h["flat"]))
    return allh[:k]


def _search_range(args):
    w, avail, kind, k, budget, min_rate, lo, hi = args
    o = Oracle(w, avail)
    return o.search(kind, k, budget=budget, min_rate=min_rate, lo=lo, hi=hi)


def parallel_search(w, kind: int, k: int, *, budget: float = 0.0, min_rate: float = 0.0, avail=None,
                    procs: int = 0, pool=None):
    """The same exhaustive pass split by flat range over worker processes (spawned)."""
    import multiprocessing as mp
    n = Oracle(w, avail).space_size()
    procs = procs or os.cpu_count() or 1
    chunks = max(procs * 8, 1)
    edges = [n * j // chunks for j in range(chunks + 1)]
    tasks = [(w, avail, kind, k, budget, min_rate, edges[j], edges[j + 1]) for j in range(chunks)]
    own = pool is None
    if own:
        pool = mp.get_context("spawn").Pool(procs)
    try:
        parts = pool.map(_search_range, tasks)
    finally:
        if own:
            pool.close()
            pool.join()
    hits = merge_hits([p[0] for p in parts], k)
    counts = {}
    for _, c in parts:
        for key, v in c.items():
            if key != "min_cost":
                counts[key] = counts.get(key, 0) + v
    costs = [c["min_cost"] for _, c in parts if c["n_feasible"]]
    counts["min_cost"] = min(costs) if costs else 0.0
    return hits, counts


def _plan_snapshot(args):
    w, snap, k = args
    o = Oracle(w, snap)
    return o.plan(k)


def plan_snapshots(w, snapshots, k: int, *, procs: int = 0, pool=None):
    """Oracle.plan for each availability snapshot of one workload, the snapshots spread over worker
    processes (spawned).  Returns a list of (hits, counts, budget), one per snapshot, in order."""
    import multiprocessing as mp
    tasks = [(w, np.array(s, dtype=np.uint16, copy=True), k) for s in snapshots]
    own = pool is None
    if own:
        pool = mp.get_context("spawn").Pool(procs or os.cpu_count() or 1)
    try:
        return pool.map(_plan_snapshot, tasks, chunksize=1)
    finally:
        if own:
            pool.close()
            pool.join()
