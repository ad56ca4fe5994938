"""Shared test helpers: fixtures -> Workload, record packing, comparisons."""
import glob
import json
import os

import numpy as np

from paper_2504_17096_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
REL_TOL_F64 = 1e-5      # the parity bar for times and costs computed in binary64


def golden_cases():
    out = []
    for path in sorted(glob.glob(os.path.join(GOLDEN, "*.json"))):
        with open(path) as f:
            out.append(json.load(f))
    return out


def workload_from_tables(t: dict, name: str = "fixture") -> W.Workload:
    """A Workload from a fixture's written-out tables, with a one-point search space."""
    f64 = lambda k: np.array(t[k], dtype=np.float64)
    u64 = lambda k: np.array(t[k], dtype=np.uint64)
    poly = {k: np.array(t[k], dtype=np.float64) for k in ("intra_bw_poly", "inter_bw_poly", "zone_bw_poly") if k in t}
    return W.Workload(
        **poly, name=name, n_blocks=t["n_blocks"], has_embed=t["has_embed"], has_head=t["has_head"],
        heads=t["heads"], gbs=t["gbs"], mul_factor=t["mul_factor"], dtype_size=t["dtype_size"],
        grad_dtype_size=t["grad_dtype_size"], tp_values=list(t["tp_values"]),
        mbs_values=list(t["mbs_values"]), fwd=f64("fwd"), bwd=f64("bwd"), upd=f64("upd"),
        params=u64("params"), act_saved=u64("act_saved"), act_ckpt=u64("act_ckpt"),
        act_work=u64("act_work"), p2p_bytes=u64("p2p_bytes"), n_types=t["n_types"],
        n_zones=t["n_zones"], capacity=u64("capacity"), reserved=u64("reserved"),
        gpus_per_node=np.array(t["gpus_per_node"], dtype=np.uint32),
        price_per_hour=f64("price_per_hour"), intra_alpha=f64("intra_alpha"),
        intra_inv_bw=f64("intra_inv_bw"), inter_alpha=f64("inter_alpha"),
        inter_inv_bw=f64("inter_inv_bw"), zone_alpha=f64("zone_alpha"), zone_inv_bw=f64("zone_inv_bw"),
        egress=f64("egress"), avail=np.array(t["avail"], dtype=np.uint16),
        p_values=[1], mbs_idx=[0], tp_idx=[0], rc_values=[0], d_values=[1], seg_max=4,
        objective=W.OBJ_MAX_THROUGHPUT)


def stages_to_records(plans):
    """Per-stage plan dicts (P, mbs_idx, rc, D, type[], zone[], tp_idx[]) -> run-length records."""
    n = len(plans)
    rec = {k: np.zeros(n, dtype=np.int64) for k in ("P", "mbs_idx", "rc", "n_runs", "D")}
    for k in ("type", "zone", "tp_idx", "n_stages"):
        rec[k] = np.zeros((n, 16), dtype=np.int64)
    for j, p in enumerate(plans):
        for k in ("P", "mbs_idx", "rc", "D"):
            rec[k][j] = p[k]
        r = -1
        prev = None
        for i in range(p["P"]):
            cur = (p["type"][i], p["zone"][i], p["tp_idx"][i])
            if cur != prev:
                r += 1
                rec["type"][j, r], rec["zone"][j, r], rec["tp_idx"][j, r] = cur
                prev = cur
            rec["n_stages"][j, r] += 1
        rec["n_runs"][j] = r + 1
    return rec


def rel_close(a, b, tol):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    both_nan = np.isnan(a) & np.isnan(b)
    scale = np.maximum(np.abs(a), np.abs(b))
    ok = np.abs(a - b) <= tol * scale
    return bool(np.all(ok | both_nan))
