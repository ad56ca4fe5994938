"""Benchmark of the plan-search hot path: candidates simulated per second and search seconds.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--impl reference]

A step is one whole search (`sailor_plan`: decode, simulate, select) over the workload's
candidate space with every candidate's time and cost evaluated (no pruning).  Rank 0 prints one
JSON line.  With --impl reference the CPU oracle is timed instead, on bounded samples.

With N > 1 ranks (one per GPU) the one space is split into contiguous flat-index ranges of equal
estimated cost, each rank searches its range with `sailor_plan_range`, and the per-rank lists are
merged by (score, flat) after one gather of k records per rank ("scaling": "strong");
`--replicas` instead gives every rank the whole space and its own availability snapshot ("weak").

Hooks for the profiling commands quoted under profiles/ (they change what is run, not how it is
timed): `--only-p P ...` keeps only those pipeline depths of the workload (a small case for ncu),
`--dp-only` runs just the dynamic-programming search, `--dp-workspace-gib` bounds its tables, `--sim-only`
runs just the explicit-batch kernels,
`--f32-screen` times the search with the binary32 screen on, `--no-cpu` / `--no-aux` drop the oracle leg / the
secondary measurements, and
`--write-counters LOG.csv` turns an ncu `--csv` log of one plan_kernel launch into the counter file
the roofline figure reads (stamped with a hash of the kernel sources it was captured on).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2504_17096_b200 import workloads as W

METRIC = "candidate plans simulated/sec"
UNIT = "candidates/s"
K_TOP = 32
# algorithmic work of one candidate with P stages, in lane operations (adds, multiplies,
# divisions, maxima, compares, table reads of the stage-by-stage evaluation)
OPS_PLAN, OPS_STAGE = 40, 35
ISSUE_PER_SM, LANES = 4, 32
# counters of one plan_kernel launch (ncu, one pass), kept with a hash of the sources they were captured on
COUNTER_FILE = os.path.join(ROOT, "profiles", "plan_kernel_cfg5_counters.txt")
COUNTER_METRICS = ("smsp__inst_executed.sum", "smsp__inst_executed_pipe_fp64.sum", "smsp__inst_executed_pipe_alu.sum",
                   "smsp__inst_executed_pipe_fma.sum", "smsp__inst_executed_pipe_lsu.sum", "dram__bytes_read.sum",
                   "dram__bytes_write.sum")
KERNEL_SOURCES = ("sailor_plan_kernels.cuh", "sailor_tables.cuh")


def kernel_source_hash() -> str:
    """Hash of the files that define plan_kernel and of the compiler flags: a counter file is only valid for
    the kernel it was captured on."""
    import hashlib
    from paper_2504_17096_b200 import build as cuda_build
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(cuda_build.CSRC, name), "rb") as f:
            h.update(f.read())
    h.update(" ".join(cuda_build.NVCC_FLAGS).encode())
    return h.hexdigest()[:16]


def read_counters(workload: str):
    """The stored counters of one plan_kernel launch on `workload`, or (None, why)."""
    try:
        with open(COUNTER_FILE) as f:
            rows = dict(line.split(None, 1) for line in f if line.strip() and not line.startswith("#"))
    except OSError:
        return None, "no counter file"
    rows = {k: v.strip() for k, v in rows.items()}
    if rows.get("workload") != workload:
        return None, f"counters are of {rows.get('workload')}"
    if rows.get("source_sha256_16") != kernel_source_hash():
        return None, "the kernel sources changed after the counters were captured"
    return {k: int(float(rows[k])) for k in COUNTER_METRICS if k in rows}, None


def write_counters(args) -> None:
    """ncu --csv log (one plan_kernel launch, the metrics of COUNTER_METRICS) -> the counter file."""
    import csv
    w = workload_by_name(args.workload, args.only_p)
    found = {}
    with open(args.write_counters, newline="") as f:
        rows = [r for r in csv.reader(f) if len(r) > 3]
    head = next(r for r in rows if "Metric Name" in r)
    i_name, i_val, i_kernel = head.index("Metric Name"), head.index("Metric Value"), head.index("Kernel Name")
    for r in rows:
        if len(r) > max(i_name, i_val) and r[i_name] in COUNTER_METRICS and "plan_kernel" in r[i_kernel]:
            found.setdefault(r[i_name], int(float(r[i_val].replace(",", ""))))
    missing = [m for m in COUNTER_METRICS if m not in found]
    if missing:
        raise SystemExit(f"the log lacks {missing}")
    with open(COUNTER_FILE, "w") as f:
        f.write("# Counters of ONE plan_kernel launch (every candidate evaluated), from one ncu pass set:\n")
        f.write("#   ncu --metrics " + ",".join(COUNTER_METRICS) + " --clock-control none -k regex:plan_kernel -c 1 \\\n")
        f.write("#       --csv --log-file LOG.csv python bench.py --steps 1 --warmup 1 --no-cpu --no-aux\n")
        f.write("#   python bench.py --write-counters LOG.csv\n")
        f.write("# bench.py uses them only while source_sha256_16 equals the hash of the kernel sources in the tree.\n")
        f.write(f"workload {w.name}\nsource_sha256_16 {kernel_source_hash()}\n")
        for m in COUNTER_METRICS:
            f.write(f"{m} {found[m]}\n")
    print(open(COUNTER_FILE).read())


def mean_ops_per_candidate(w: W.Workload) -> float:
    base = len(w.mbs_idx) * len(w.tp_idx) * len(w.rc_values) * len(w.d_values)
    tot = ops = 0
    for p in w.p_values:
        n = base * w.radix ** min(p, w.seg_max)
        tot += n
        ops += n * (OPS_PLAN + OPS_STAGE * p)
    return ops / tot


def workload_by_name(name: str, only_p=None) -> W.Workload:
    w = W.CONFIGS[int(name.replace("cfg", ""))]()
    if only_p:                       # a sub-space with the given stage counts only (small profiling cases)
        w.p_values = [p for p in w.p_values if p in only_p]
        w.name += "-P" + "_".join(str(p) for p in w.p_values)
    return w


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "10"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            pass

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        # the sampler runs only while the timed regions run, so every sample is under load
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "samples": len(sm), "reasons": sorted(reasons)}


def run_reference(args) -> None:
    """The CPU oracle, as it stands, on bounded samples of the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle.binding import Oracle
    w = workload_by_name(args.workload, args.only_p)
    o = Oracle(w)
    n = o.space_size()
    sample = min(n, args.ref_sample)
    stride = max(1, n // sample)
    times, done = [], 0
    for step in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        _, counts = o.search(w.objective, K_TOP, lo=step % stride, stride=stride)
        dt = time.perf_counter() - t0
        if step >= args.warmup:
            times.append(dt)
            done += counts["n_total"]
    value = done / sum(times)
    desc = f"every {stride}-th flat index of {w.name} ({done // max(1, args.steps)} candidates per step)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "candidates": n, "sampled": True},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def pruning_modes(B, ctx, w, sp) -> dict:
    """The planner's pruning heuristics as search modes (degree order with early termination, smallest
    fitting tensor-parallel degree): search seconds, how much was left out, and whether the best plan
    is still the exhaustive search's."""
    full, _ = B.sailor_plan(ctx, sp, B.make_objective(w), 1)
    modes = {"min_tp_only": B.FLAG_MIN_TP_ONLY}
    if w.objective in (W.OBJ_MAX_THROUGHPUT, W.OBJ_MIN_COST):
        modes["degree_order"] = B.FLAG_DEGREE_ORDER
        modes["degree_order+min_tp_only"] = B.FLAG_DEGREE_ORDER | B.FLAG_MIN_TP_ONLY
    out = {}
    for name, flags in modes.items():
        ob = B.make_objective(w, flags=flags)
        B.sailor_plan(ctx, sp, ob, K_TOP)
        ts = []
        for _ in range(5):
            t0 = time.perf_counter()
            B.sailor_set_availability(ctx, w.avail)
            res, st = B.sailor_plan(ctx, sp, ob, K_TOP)
            ts.append(time.perf_counter() - t0)
        out[name] = {"search_s": statistics.median(ts), "kernel_ms": st.kernel_ms, "launches": int(st.n_launches),
                     "looked_at": int(st.n_total), "skipped": int(st.n_skipped), "pruned_tp": int(st.n_pruned_tp),
                     "configs_evaluated": int(st.n_configs_evaluated), "configs": int(st.n_configs),
                     "feasible": int(st.n_feasible),
                     "same_best_as_exhaustive": bool(res and full and res[0].flat == full[0].flat),
                     "score_over_exhaustive": (res[0].score / full[0].score) if (res and full) else None}
    return out


def dp_search(B, ctx, w, sp) -> dict:
    """Per-stage GPU types by the dynamic-programming recursion (one zone order: zones as numbered),
    next to the best iteration time the segment search finds in its own space."""
    orders = [list(range(w.n_zones))]
    B.sailor_plan_dp(ctx, sp, orders, K_TOP)
    ts = []
    for _ in range(3):
        t0 = time.perf_counter()
        B.sailor_set_availability(ctx, w.avail)
        res, st = B.sailor_plan_dp(ctx, sp, orders, K_TOP)
        ts.append(time.perf_counter() - t0)
    seg, _ = B.sailor_plan(ctx, sp, B.make_objective(w, kind=W.OBJ_MAX_THROUGHPUT, budget=0.0, min_rate=0.0, factor=0.0), 1)
    # bytes the level kernel must move per table entry: its value (32 B) and choice (1 B) written once
    return {"search_s": statistics.median(ts), "kernel_ms": st.kernel_ms, "problems": int(st.n_problems),
            "solved": int(st.n_solved), "table_entries": int(st.n_states), "batches": int(st.n_batches),
            "launches": int(st.n_launches), "workspace_bytes": int(st.workspace_used),
            "entries_per_s": st.n_states / (st.kernel_ms / 1e3) if st.kernel_ms > 0 else None,
            "write_gb_per_s": st.n_states * 33 / (st.kernel_ms / 1e3) / 1e9 if st.kernel_ms > 0 else None,
            "best_t_iter": res[0].t_iter if res else None, "best_stages": int(res[0].P) if res else None,
            "segment_search_best_t_iter": seg[0].t_iter if seg else None}


def cold_search(B, torch, dev, w, flags: int = 0) -> dict:
    """What a planner invoked once per job pays: a fresh context (tables uploaded, per-composition sums formed)
    and its first search of the space (index arrays, survey, per-configuration table cache), wall clock."""
    t0 = time.perf_counter()
    ctx = B.sailor_create(w, dev, torch.cuda.current_stream().cuda_stream)
    try:
        B.sailor_set_availability(ctx, w.avail)
        t1 = time.perf_counter()
        res, _ = B.sailor_plan(ctx, B.make_space(w), B.make_objective(w, flags=flags), K_TOP)
        t2 = time.perf_counter()
    finally:
        B.sailor_destroy(ctx)
    return {"create_s": t1 - t0, "first_search_s": t2 - t1, "cold_search_s": t2 - t0, "found": len(res)}


def dp_budget_loop(B, ctx, w, budget: float) -> dict:
    """The per-stage recursion steered by the budget (Sec. 4.2.3) next to the plain check of the budget on the
    unlimited recursion's plans: workload 2 with pipelines of up to 8 stages, every zone order."""
    sub = W.config2()
    sub.p_values = [p for p in sub.p_values if p <= 8]
    sp = B.make_space(sub)
    orders = B.all_zone_orders(sub.n_zones)
    out = {"budget": budget, "problems": None}
    for name, loop in (("check_only", False), ("budget_loop", True)):
        B.sailor_plan_dp(ctx, sp, orders, K_TOP, budget=budget, budget_loop=loop)
        ts = []
        for _ in range(3):
            t0 = time.perf_counter()
            res, st = B.sailor_plan_dp(ctx, sp, orders, K_TOP, budget=budget, budget_loop=loop)
            ts.append(time.perf_counter() - t0)
        out["problems"] = int(st.n_problems)
        out[name] = {"search_s": statistics.median(ts), "kernel_ms": st.kernel_ms, "with_a_plan": int(st.n_solved),
                     "within_budget": int(st.n_solved - st.n_over_constraint), "unfinished": int(st.n_unfinished),
                     "calls_or_entries": int(st.n_states), "best_t_iter": res[0].t_iter if res else None}
    return out


def mixed_search(B, ctx, w) -> dict:
    """Search over plans whose stages mix GPU types among their replicas: workload 2's model and cluster, two
    pipeline depths, replicas split in quarters, next to the same space with one type per stage."""
    sub = W.config2()
    sub.p_values, sub.mbs_idx, sub.d_values = [2, 4], [sub.mbs_idx[1]], [4, 8]
    tps = [0, 1, 2]
    obj = B.Objective(W.OBJ_MAX_THROUGHPUT, 0, 0.0, 0.0, 0.0)
    out = {}
    for name, gran in (("one_type_per_stage", 1), ("quarters", 4)):
        sp = B.make_mixed_space(sub, gran, tps)
        B.sailor_plan_mixed(ctx, sp, obj, K_TOP)
        ts = []
        for _ in range(3):
            t0 = time.perf_counter()
            res, st = B.sailor_plan_mixed(ctx, sp, obj, K_TOP)
            ts.append(time.perf_counter() - t0)
        out[name] = {"candidates": int(st.n_total), "feasible": int(st.n_feasible), "search_s": statistics.median(ts),
                     "kernel_ms": st.kernel_ms, "plans_per_s": st.n_total / (st.kernel_ms / 1e3),
                     "best_t_iter": res[0].t_iter if res else None,
                     "best_mixes_types": bool(res and any(s.n_groups > 1 for s in res[0].plan.stage[: res[0].plan.P]))}
    return out


def explicit_batches(B, torch, dev) -> dict:
    """sailor_simulate / sailor_simulate_mixed on batches resident in HBM (larger than L2), CUDA events."""
    out = {}
    # explicit batches (sailor_simulate) with records resident in HBM: 72 B in + 28 B out per plan
    w = W.config5()
    ctx = B.sailor_create(w, dev, torch.cuda.current_stream().cuda_stream)
    try:
        B.sailor_set_availability(ctx, w.avail)
        sp5 = B.make_space(w)
        n5 = B.sailor_space_size(ctx, sp5)
        rng = W.SplitMix64(12)
        enumerated = np.zeros(1 << 15, dtype=B.REC_DTYPE)              # records of the search space itself
        for j in range(enumerated.size):
            rec = B.sailor_decode(ctx, sp5, rng.next_u64() % n5)
            enumerated[j] = np.frombuffer(bytes(rec), dtype=B.REC_DTYPE)[0]
        batches = {"simulate_cfg5_records": B.pack_records(W.random_plans(w, 1 << 15, seed=11, hetero_tp=True)),
                   "simulate_cfg5_enumerated": enumerated}
        for key, base in batches.items():
            reps = 128
            n = base.size * reps                                       # 4.2e6 records, 302 MB: larger than L2
            d_plans = torch.from_numpy(base.view(np.uint8).reshape(-1, 72).copy()).cuda().repeat(reps, 1).contiguous()
            t = torch.empty(n, dtype=torch.float64, device="cuda")
            c = torch.empty(n, dtype=torch.float64, device="cuda")
            m = torch.empty(n, dtype=torch.int64, device="cuda")
            st = torch.empty(n, dtype=torch.int32, device="cuda")
            call = lambda: B.sailor_simulate_device(ctx, d_plans.data_ptr(), n, t.data_ptr(), m.data_ptr(),
                                                    c.data_ptr(), st.data_ptr())
            for _ in range(3):
                call()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(5):
                call()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / 5
            mean_p = float(base["P"].astype(np.float64).mean())
            out[key] = {"plans": n, "mean_stages": mean_p, "kernel_ms": ms, "plans_per_s": n / ms * 1e3,
                        "hbm_gb_per_s": n * 100 / ms / 1e6}
            # the same batch through the host path: records and results in pinned host memory, copies inside the call
            h_plans = d_plans.cpu().pin_memory()
            ht = torch.empty(n, dtype=torch.float64).pin_memory(); hc = torch.empty(n, dtype=torch.float64).pin_memory()
            hm = torch.empty(n, dtype=torch.int64).pin_memory(); hs = torch.empty(n, dtype=torch.int32).pin_memory()
            host_call = lambda: B.sailor_simulate_host(ctx, h_plans.data_ptr(), n, ht.data_ptr(), hm.data_ptr(),
                                                       hc.data_ptr(), hs.data_ptr())
            host_call()
            ts = []
            for _ in range(3):
                t0 = time.perf_counter()
                host_call()
                ts.append(time.perf_counter() - t0)
            torch.cuda.synchronize()
            same = bool(torch.equal(ht.view(torch.int64), t.cpu().view(torch.int64)) and torch.equal(hs, st.cpu()))
            out[key].update({"host_call_ms": statistics.median(ts) * 1e3, "host_plans_per_s": n / statistics.median(ts),
                             "host_pcie_gb_per_s": n * 100 / statistics.median(ts) / 1e9, "host_equals_device": same})
            del d_plans, t, c, m, st, h_plans, ht, hc, hm, hs
        # plans whose stages mix GPU types among their replicas, up to 32 stages each: 648 B in + 28 B out per plan
        base = B.pack_mixed_plans(W.random_mixed_plans(w, 1 << 14, seed=13), stages=32)
        reps = 64
        n = base.size * reps                                           # 1.05e6 plans, 680 MB: larger than L2
        d_plans = torch.from_numpy(base.view(np.uint8).reshape(-1, base.itemsize).copy()).cuda().repeat(reps, 1).contiguous()
        t = torch.empty(n, dtype=torch.float64, device="cuda")
        c = torch.empty(n, dtype=torch.float64, device="cuda")
        m = torch.empty(n, dtype=torch.int64, device="cuda")
        st = torch.empty(n, dtype=torch.int32, device="cuda")
        call = lambda: B.sailor_simulate_mixed_device(ctx, d_plans.data_ptr(), n, t.data_ptr(), m.data_ptr(),
                                                      c.data_ptr(), st.data_ptr(), record_bytes=base.itemsize)
        for _ in range(3):
            call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(5):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 5
        out["simulate_mixed_cfg5"] = {"plans": n, "mean_stages": float(base["P"].astype(np.float64).mean()),
                                      "kernel_ms": ms, "plans_per_s": n / ms * 1e3,
                                      "hbm_gb_per_s": n * (base.itemsize + 28) / ms / 1e6}
        del d_plans, t, c, m, st
    finally:
        B.sailor_destroy(ctx)
    return out


def aux_measurements(B, torch, dev, oracle_cfg4=None) -> dict:
    """Search seconds of the other workloads through the public call (host buffers), default mode."""
    out = {}
    for cfg in (1, 2, 3, 6):
        w = W.CONFIGS[cfg]()
        cold = cold_search(B, torch, dev, w)
        ctx = B.sailor_create(w, dev, torch.cuda.current_stream().cuda_stream)
        try:
            sp, ob = B.make_space(w), B.make_objective(w)
            B.sailor_set_availability(ctx, w.avail)
            B.sailor_plan(ctx, sp, ob, K_TOP)
            ts = []
            for _ in range(5):
                t0 = time.perf_counter()
                B.sailor_set_availability(ctx, w.avail)
                _, st = B.sailor_plan(ctx, sp, ob, K_TOP)
                ts.append(time.perf_counter() - t0)
            out[f"cfg{cfg}"] = {"candidates": int(st.n_total), "search_s": statistics.median(ts),
                                "kernel_ms": st.kernel_ms, "h2d_ms": st.h2d_ms, "d2h_ms": st.d2h_ms,
                                "launches": int(st.n_launches), "passes": 2 if w.budget_factor_over_cheapest > 0 else 1,
                                "cold_search_s": cold["cold_search_s"], "cold": cold}
            out[f"cfg{cfg}"]["pruning_modes"] = pruning_modes(B, ctx, w, sp)
            out[f"cfg{cfg}"]["dp"] = dp_search(B, ctx, w, sp)
            if cfg == 2:
                out["cfg2"]["dp_budget_loop"] = dp_budget_loop(B, ctx, w, st.budget_used)
                out["cfg2"]["mixed_search"] = mixed_search(B, ctx, w)
        finally:
            B.sailor_destroy(ctx)
    out.update(explicit_batches(B, torch, dev))
    w = W.config4()
    ctx = B.sailor_create(w, dev, torch.cuda.current_stream().cuda_stream)
    try:
        sp, ob = B.make_space(w), B.make_objective(w)
        B.sailor_set_availability(ctx, w.snapshots[0])
        B.sailor_plan(ctx, sp, ob, 4)
        lat, best = [], []
        for snap in w.snapshots:
            t0 = time.perf_counter()
            B.sailor_set_availability(ctx, snap)
            res, _ = B.sailor_plan(ctx, sp, ob, 4)
            lat.append(time.perf_counter() - t0)
            best.append(int(res[0].flat) if res else None)
        lat.sort()
        out["cfg4"] = {"snapshots": len(lat), "replan_p50_s": lat[len(lat) // 2], "replan_p99_s": lat[int(len(lat) * 0.99)],
                       "replan_max_s": lat[-1]}
        if oracle_cfg4 is not None:        # best-plan agreement with the oracle's two-pass plan of every snapshot
            want = [(h[0]["flat"] if h else None) for h, _, _ in oracle_cfg4["plans"]]
            out["cfg4"]["agree"] = f"{sum(int(a == b) for a, b in zip(best, want))}/{len(want)}"
            out["cfg4"]["oracle_s_per_snapshot"] = oracle_cfg4["core_s"] / len(want)
            out["cfg4"]["oracle_cores"] = oracle_cfg4["cores"]
    finally:
        B.sailor_destroy(ctx)
    return out


def run_sim_only(args) -> None:
    """Only the explicit-batch kernels (a few hundred MB on the device): a small command for profiling them.
    Prints one JSON line of its own (not the benchmark line)."""
    import torch
    from paper_2504_17096_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    print(json.dumps({"sim_only": explicit_batches(B, torch, 0)}), flush=True)


def run_dp_only(args) -> None:
    """Only the dynamic-programming search of the workload (one zone order), a few times: a small command for
    profiling its kernels.  Prints one JSON line of its own (not the benchmark line)."""
    import torch
    from paper_2504_17096_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    w = workload_by_name(args.workload, args.only_p)
    ctx = B.sailor_create(w, 0, torch.cuda.current_stream().cuda_stream)
    try:
        B.sailor_set_availability(ctx, w.avail)
        sp = B.make_space(w)
        orders = [list(range(w.n_zones))]
        for _ in range(max(1, args.steps)):
            t0 = time.perf_counter()
            res, st = B.sailor_plan_dp(ctx, sp, orders, K_TOP, workspace_bytes=int(args.dp_workspace_gib * (1 << 30)))
            dt = time.perf_counter() - t0
        print(json.dumps({"dp_only": w.name, "search_s": dt, "kernel_ms": st.kernel_ms, "problems": int(st.n_problems),
                          "solved": int(st.n_solved), "table_entries": int(st.n_states), "batches": int(st.n_batches),
                          "launches": int(st.n_launches), "workspace_bytes": int(st.workspace_used),
                          "best_t_iter": res[0].t_iter if res else None}), flush=True)
    finally:
        B.sailor_destroy(ctx)


def oracle_cfg4_plans() -> dict:
    """The oracle's two-pass plan of each of workload 4's 200 snapshots, spread over the host cores (spawned
    workers), for the best-plan agreement count."""
    from oracle.binding import plan_snapshots
    w = W.config4()
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    plans = plan_snapshots(w, w.snapshots, 1, procs=cores)
    dt = time.perf_counter() - t0
    return {"plans": plans, "cores": cores, "wall_s": dt, "core_s": dt * min(cores, len(plans))}


def run_ours(args) -> None:
    import torch
    from paper_2504_17096_b200 import binding as B
    from paper_2504_17096_b200 import build as cuda_build
    from paper_2504_17096_b200 import sharding
    if cuda_build.is_stale():                    # compile the CUDA library if it is missing or out of date
        if int(os.environ.get("LOCAL_RANK", "0")) == 0:
            cuda_build.build()
        else:                                    # one rank per node builds, the others wait for the file
            deadline = time.time() + 300
            while cuda_build.is_stale() and time.time() < deadline:
                time.sleep(0.5)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    # one rank per GPU over NCCL; for a dry run of the multi-rank control flow on fewer GPUs than
    # ranks (the searches are independent, no rank waits for another rank's kernel) the environment
    # may select the gloo backend and let ranks share devices
    backend = os.environ.get("SAILOR_BENCH_BACKEND", "nccl")
    if os.environ.get("SAILOR_BENCH_SHARE_GPUS"):
        local %= torch.cuda.device_count()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)

    w = workload_by_name(args.workload, args.only_p)
    # one space split over the ranks by flat-index range, unless asked for replicas (or the workload's budget
    # rule needs the cheapest plan of the whole space first)
    split = world > 1 and not args.replicas and not w.budget_factor_over_cheapest > 0
    avail = w.avail.copy()
    if rank and not split:               # replicas: every rank searches the whole space for its own snapshot
        rng = W.SplitMix64(0xA7A11 + rank)
        for idx in np.ndindex(avail.shape):
            avail[idx] = min(65535, max(0, int(avail[idx]) + rng.randint(0, 8) - 4))
    stream = torch.cuda.current_stream()
    ctx = B.sailor_create(w, local, stream.cuda_stream)
    space = B.make_space(w)
    obj = B.make_objective(w, flags=B.FLAG_EVAL_ALL | (B.FLAG_F32_SCREEN if args.f32_screen else 0))
    n = B.sailor_space_size(ctx, space)
    lo, hi = (sharding.split_by_cost(sharding.subspace_costs(w), world, rank) if split else (0, n))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # larger than the 126 MB L2

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def search():
        return B.sailor_plan_range(ctx, space, obj, lo, hi, K_TOP) if split else B.sailor_plan(ctx, space, obj, K_TOP)

    def merged(res, st):
        """The job's result: this rank's list, or the lists of all ranges merged by (score, flat)."""
        if not split:
            return [(r.score, int(r.flat)) for r in res], int(st.n_total)
        counts = {"n_total": int(st.n_total), "n_feasible": int(st.n_feasible), "min_feasible_cost": st.min_feasible_cost}
        top, tot = sharding.gather_and_merge([(r.score, int(r.flat)) for r in res], counts, K_TOP)
        return top, tot["n_total"]

    split_check = None
    if split:      # the split must reproduce a single search: checked on a small workload before anything is timed
        small = W.config1()
        c1 = B.sailor_create(small, local, stream.cuda_stream)
        try:
            B.sailor_set_availability(c1, small.avail)
            sp1, ob1 = B.make_space(small), B.make_objective(small)
            a, b = sharding.split_range(B.sailor_space_size(c1, sp1), world, rank)
            part, pst = B.sailor_plan_range(c1, sp1, ob1, a, b, K_TOP)
            top, _ = sharding.gather_and_merge([(r.score, int(r.flat)) for r in part], {"n_total": int(pst.n_total)}, K_TOP)
            whole, _ = B.sailor_plan(c1, sp1, ob1, K_TOP)
            split_check = top == [(r.score, int(r.flat)) for r in whole]
            assert split_check, "the merged per-range lists differ from the single search"
        finally:
            B.sailor_destroy(c1)

    B.sailor_set_availability(ctx, avail)
    for _ in range(args.warmup):
        search()

    # ---- device-timed region: inputs resident, CUDA events on the launching stream ------------
    barrier()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid)) if rank == 0 else None
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    kernel_ms, launches, res, st = [], 0, [], None
    for a, b in ev:
        flush.fill_(1)                                   # L2 flush between timed iterations
        a.record(stream)
        res, st = search()
        b.record(stream)
        kernel_ms.append(st.kernel_ms)
        launches += st.n_launches
    barrier()
    step_ms = [a.elapsed_time(b) for a, b in ev]
    dev_s = sum(step_ms) / 1e3
    top, n_seen = merged(res, st)

    # ---- end to end: the public call with host buffers (availability up, results down; with several ranks
    # ---- also the exchange and merge of the per-range lists) -----------------------------------------
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        B.sailor_set_availability(ctx, avail)
        res, st = search()
        merged(res, st)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    clocks = sampler.stop() if sampler else None          # samples of both timed regions
    h2d = int(avail.size * 2)
    d2h = int(K_TOP * 120 + 96)

    times = torch.tensor([dev_s, e2e_s], dtype=torch.float64, device="cuda" if backend == "nccl" else "cpu")
    if dist is not None:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    dev_s, e2e_s = (float(x) for x in times.cpu())
    total = n * args.steps * (1 if split else world)
    if split:
        assert n_seen == n, "the ranges do not add up to the space"

    if rank == 0:
        ops = mean_ops_per_candidate(w)
        k_s = statistics.mean(kernel_ms) / 1e3
        peaks = {}
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                peaks = json.load(f)
        except OSError:
            pass
        # the ceiling: what the device really issues, measured now with three instruction streams
        rates = B.sailor_measure_issue_rates(local, stream.cuda_stream, 5)
        sm_max = float(peaks.get("sm_max_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0)
        units_x_clock = rates.sm_count * ISSUE_PER_SM * sm_max * 1e6                 # warp-instructions/s
        counters, why_not = (read_counters(w.name) if world == 1 and not args.f32_screen
                             else (None, "counters are of a whole-space launch of the binary64 search"))
        roofline = {"bound": "alu", "unit": "warp-inst/s", "achieved": None, "peak": rates.ffma_warp_inst_per_s,
                    "frac": None, "traffic": None,
                    "peak_kind": "measured: FP32 multiply-add stream, 8 chains per thread, 4 x 256 threads per SM",
                    "peak_units_x_clock": units_x_clock, "frac_of_units_x_clock": None,
                    "issue_peak_measured": {"ffma": rates.ffma_warp_inst_per_s, "imad": rates.imad_warp_inst_per_s,
                                            "dadd": rates.dadd_warp_inst_per_s,
                                            "per_sm_per_cycle_at_max_clock": {
                                                k: v / (rates.sm_count * sm_max * 1e6) for k, v in
                                                (("ffma", rates.ffma_warp_inst_per_s), ("imad", rates.imad_warp_inst_per_s),
                                                 ("dadd", rates.dadd_warp_inst_per_s))}},
                    "fp64_achieved": None, "fp64_peak": rates.dadd_warp_inst_per_s, "fp64_frac": None,
                    "lane_inst_per_candidate": None, "counters": why_not or os.path.relpath(COUNTER_FILE, ROOT),
                    "algorithmic_over_peak": ops * n / k_s / (units_x_clock * LANES),
                    "ops_per_candidate_model": ops, "kernel_ms": 1e3 * k_s,
                    "note": "achieved = warp-instructions one plan_kernel launch executes (ncu smsp__inst_executed.sum, "
                            "stored with a hash of the kernel sources) / this run's kernel time; fp64_* = the same for the "
                            "FP64 pipe against the FP64-add stream; algorithmic_over_peak = (40 + 35 P lane-ops per "
                            "candidate) / kernel time over units x clock: above 1 because prefix sums and run-length "
                            "segments remove most of the stage-by-stage work"}
        if counters:
            inst, fp64 = counters["smsp__inst_executed.sum"], counters["smsp__inst_executed_pipe_fp64.sum"]
            roofline.update(achieved=inst / k_s, frac=inst / k_s / rates.ffma_warp_inst_per_s,
                            frac_of_units_x_clock=inst / k_s / units_x_clock,
                            traffic=counters["dram__bytes_read.sum"] + counters["dram__bytes_write.sum"],
                            fp64_achieved=fp64 / k_s, fp64_frac=fp64 / k_s / rates.dadd_warp_inst_per_s,
                            lane_inst_per_candidate=inst * LANES / n,
                            pipe_share={k.split("pipe_")[1].split(".")[0]: counters[k] / inst for k in counters if "pipe_" in k})
        cpu, oracle4 = None, None
        if world == 1 and not args.no_cpu:
            from oracle.binding import Oracle
            o = Oracle(w)
            sample = min(n, args.cpu_sample)
            stride = max(1, n // sample)
            t0 = time.perf_counter()
            _, counts = o.search(w.objective, K_TOP, stride=stride)
            dt = time.perf_counter() - t0
            cpu = {"value": counts["n_total"] / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                   "sample": f"every {stride}-th flat index of {w.name}: {counts['n_total']} candidates in {dt:.1f} s"}
            if not args.no_aux:
                oracle4 = oracle_cfg4_plans()
        aux = aux_measurements(B, torch, local, oracle4) if (world == 1 and not args.no_aux) else None
        if aux is not None:
            # the same workload the way a planner would call it: memory/availability pruning on
            ob = B.make_objective(w)
            ts = []
            for _ in range(5):
                t0 = time.perf_counter()
                B.sailor_set_availability(ctx, avail)
                _, stp = B.sailor_plan(ctx, space, ob, K_TOP)
                ts.append(time.perf_counter() - t0)
            aux[args.workload + "_default_mode"] = {"candidates": int(stp.n_total), "search_s": statistics.median(ts),
                                                    "kernel_ms": stp.kernel_ms, "feasible": int(stp.n_feasible),
                                                    "cold": cold_search(B, torch, local, w),
                                                    "pruning_modes": pruning_modes(B, ctx, w, space),
                                                    "dp": dp_search(B, ctx, w, space)}
            aux[args.workload + "_every_candidate"] = {"cold": cold_search(B, torch, local, w, B.FLAG_EVAL_ALL)}
            # the same search with the binary32 screen: identical results, the second figure
            obs = B.make_objective(w, flags=B.FLAG_EVAL_ALL | B.FLAG_F32_SCREEN)
            for _ in range(3):
                B.sailor_plan(ctx, space, obs, K_TOP)
            km = []
            for _ in range(10):
                flush.fill_(1)
                rs, sts = B.sailor_plan(ctx, space, obs, K_TOP)
                km.append(sts.kernel_ms)
            aux[args.workload + "_f32_screen"] = {
                "kernel_ms": statistics.median(km), "candidates_per_s": n / (statistics.median(km) / 1e3),
                "same_results": [(r.flat, r.score) for r in rs] == [(int(f), sc) for sc, f in top] if not split else None}
        line = {"metric": METRIC, "value": total / dev_s, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": 1e3 * dev_s / args.steps, "higher_is_better": True,
                "scaling": "strong" if split else "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": w.name, "candidates": n, "top_k": K_TOP,
                           "mode": "every candidate evaluated" + (" (binary32 screen, binary64 re-score)" if args.f32_screen else ""),
                           "objective": w.objective, "l2": "flushed between timed iterations (256 MiB write)",
                           "parallelism": ("1 gpu" if world == 1 else
                                           f"one space split into {world} flat-index ranges of equal estimated cost, "
                                           f"top-{K_TOP} lists merged" if split else f"{world} independent searches"),
                           "split_check": split_check},
                "e2e": {"value": total / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "search_s": e2e_s / args.steps, "h2d_ms": st.h2d_ms, "d2h_ms": st.d2h_ms},
                "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu,
                "best": None if not top else {"flat": top[0][1], "score": top[0][0]},
                "aux": aux}
        print(json.dumps(line), flush=True)
    B.sailor_destroy(ctx)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg5")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-sample", type=int, default=20_000_000, help="candidates the CPU baseline evaluates")
    ap.add_argument("--ref-sample", type=int, default=4_000_000, help="candidates per reference step")
    ap.add_argument("--only-p", type=int, nargs="*", default=None, help="keep only these pipeline depths")
    ap.add_argument("--dp-only", action="store_true", help="run only the dynamic-programming search (for profiling)")
    ap.add_argument("--sim-only", action="store_true", help="run only the explicit-batch kernels (for profiling)")
    ap.add_argument("--dp-workspace-gib", type=float, default=8.0, help="table workspace of --dp-only")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-aux", action="store_true")
    ap.add_argument("--f32-screen", action="store_true", help="time the search with the binary32 screen on (for profiling)")
    ap.add_argument("--replicas", action="store_true", help="N > 1: every rank searches the whole space (weak scaling)")
    ap.add_argument("--write-counters", default=None, metavar="NCU_CSV", help="write the counter file from an ncu --csv log")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.write_counters:
        write_counters(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.dp_only:
        run_dp_only(args)
    elif args.sim_only:
        run_sim_only(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
