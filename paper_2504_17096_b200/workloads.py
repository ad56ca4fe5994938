"""Seeded synthetic workloads: model, per-layer profile, cluster, search space, objective.

These are *inputs*.  Nothing here simulates a plan: the module only fills the tables that
the simulator consumes (Sailor Sec. 4.1 describes what the profiler would have measured:
per-layer forward/backward/update time per GPU type, microbatch size and tensor-parallel
degree, parameter counts, activation bytes, and link bandwidths) with numbers of realistic
shape, from one counter-based generator, so that two independent implementations can be
fed exactly the same arrays.

The five workloads stand in for the paper's OPT-350M / GPT-Neo-2.7B profiles on A100/V100
clusters and its geo-distributed setups (Sec. 5), which cannot be measured here.

Randomness: SplitMix64 (Steele, Lea, Flood 2014) -> 53-bit uniforms; normals by
Box-Muller; Poisson by inversion of the cumulative mass function.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

EMBED, BLOCK, HEAD = 0, 1, 2
KINDS = 3
GIB = 1 << 30
MASK64 = (1 << 64) - 1

OBJ_MAX_THROUGHPUT = 0
OBJ_MIN_COST = 1
OBJ_MAX_THROUGHPUT_PER_USD = 2


class SplitMix64:
    """Counter-based 64-bit generator; every draw advances the state by one constant."""

    def __init__(self, seed: int):
        self.state = seed & MASK64

    def next_u64(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & MASK64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
        return z ^ (z >> 31)

    def uniform(self) -> float:
        """Uniform in [0, 1) with 53 random bits."""
        return (self.next_u64() >> 11) * (1.0 / (1 << 53))

    def randint(self, lo: int, hi: int) -> int:
        """Uniform integer in [lo, hi] (modulo bias is irrelevant at these ranges)."""
        return lo + self.next_u64() % (hi - lo + 1)

    def normal(self) -> float:
        u1 = 1.0 - self.uniform()          # (0, 1]
        u2 = self.uniform()
        return math.sqrt(-2.0 * math.log(u1)) * math.cos(2.0 * math.pi * u2)

    def lognormal(self, mu: float, sigma: float) -> float:
        return math.exp(mu + sigma * self.normal())

    def poisson(self, lam: float) -> int:
        u = self.uniform()
        k = 0
        p = math.exp(-lam)
        c = p
        while u > c and k < 10_000:
            k += 1
            p *= lam / k
            c += p
        return k


@dataclass
class Workload:
    """All inputs of one search, as plain numbers and numpy arrays (C order)."""

    name: str
    # model
    n_blocks: int
    has_embed: int
    has_head: int
    heads: int
    gbs: int
    mul_factor: int
    dtype_size: int
    grad_dtype_size: int
    # profile
    tp_values: List[int]
    mbs_values: List[int]
    fwd: np.ndarray          # f64 [kind][type][tp][mbs]
    bwd: np.ndarray          # f64 [kind][type][tp][mbs]
    upd: np.ndarray          # f64 [kind][type][tp]
    params: np.ndarray       # u64 [kind]
    act_saved: np.ndarray    # u64 [kind][tp][mbs]
    act_ckpt: np.ndarray     # u64 [kind][tp][mbs]
    act_work: np.ndarray     # u64 [kind][tp][mbs]
    p2p_bytes: np.ndarray    # u64 [mbs]
    # cluster
    n_types: int
    n_zones: int
    capacity: np.ndarray         # u64 [type]
    reserved: np.ndarray         # u64 [type]
    gpus_per_node: np.ndarray    # u32 [type]
    price_per_hour: np.ndarray   # f64 [zone][type]
    intra_alpha: np.ndarray      # f64 [zone][type]
    intra_inv_bw: np.ndarray     # f64 [zone][type]
    inter_alpha: np.ndarray      # f64 [zone][type]
    inter_inv_bw: np.ndarray     # f64 [zone][type]
    zone_alpha: np.ndarray       # f64 [zone][zone]
    zone_inv_bw: np.ndarray      # f64 [zone][zone]
    egress: np.ndarray           # f64 [zone][zone]
    avail: np.ndarray            # u16 [zone][type]
    # space
    p_values: List[int]
    mbs_idx: List[int]
    tp_idx: List[int]
    rc_values: List[int]
    d_values: List[int]
    seg_max: int
    # objective
    objective: int
    budget_usd_per_iter: float = 0.0
    min_iters_per_s: float = 0.0
    budget_factor_over_cheapest: float = 0.0
    # optional fitted bandwidth polynomials (bytes/s as a cubic in the message size); None = inv_bw is used
    intra_bw_poly: Optional[np.ndarray] = None   # f64 [zone][type][4]
    inter_bw_poly: Optional[np.ndarray] = None   # f64 [zone][type][4]
    zone_bw_poly: Optional[np.ndarray] = None    # f64 [zone][zone][4]
    # dynamic availability (workload 4): [snapshot][zone][type]
    snapshots: Optional[np.ndarray] = None
    notes: Dict[str, float] = field(default_factory=dict)

    @property
    def radix(self) -> int:
        return self.n_types * self.n_zones

    def space_size(self) -> int:
        """Candidate count, from the radices alone (a closed form, not an enumeration)."""
        base = len(self.mbs_idx) * len(self.tp_idx) * len(self.rc_values) * len(self.d_values)
        return sum(base * self.radix ** min(p, self.seg_max) for p in self.p_values)


def _inv_bw(gb_per_s: float) -> float:
    return 1.0 / (gb_per_s * 1e9)


def _ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def make_workload(name: str, *, seed: int, L: int, h: int, a: int, s: int, V: int, gbs: int,
                  type_mem_gib: List[int], type_base: List[float], type_price: List[float],
                  n_zones: int, gpus_per_node: int, intra_gbs: float, inter_gbs: float,
                  zone_bw_fn, avail_fn, tp_values: List[int], mbs_values: List[int],
                  p_values: List[int], d_values: List[int], rc_values: List[int],
                  objective: int, budget_factor: float = 0.0, seg_max: int = 4,
                  alpha: float = 0.0, egress_usd_per_byte: float = 1e-11) -> Workload:
    """Fill every table of one workload from `seed`.

    Time tables: BLOCK forward = base[type] * mbs^0.9 / tp^0.85 * lognormal(0, 0.05), one
    draw per (type, tp, mbs); backward = 2 x an independently drawn forward entry; HEAD =
    BLOCK x V / (12 h + 2 s) (flop ratio); EMBED = 0.02 x BLOCK; update = 0.3 base / tp per
    BLOCK, other kinds in proportion to their parameter count.
    """
    rng = SplitMix64(seed)
    T, Z = len(type_mem_gib), n_zones
    n_tp, n_mbs = len(tp_values), len(mbs_values)

    params = np.zeros(KINDS, dtype=np.uint64)
    params[EMBED] = V * h + s * h
    params[BLOCK] = 12 * h * h + 13 * h
    params[HEAD] = V * h

    fwd = np.zeros((KINDS, T, n_tp, n_mbs))
    bwd = np.zeros((KINDS, T, n_tp, n_mbs))
    upd = np.zeros((KINDS, T, n_tp))
    head_ratio = V / (12.0 * h + 2.0 * s)
    for g in range(T):
        for ti, tp in enumerate(tp_values):
            for mi, mbs in enumerate(mbs_values):
                shape = type_base[g] * math.pow(mbs, 0.9) / math.pow(tp, 0.85)
                f = shape * rng.lognormal(0.0, 0.05)
                b = 2.0 * shape * rng.lognormal(0.0, 0.05)
                fwd[BLOCK, g, ti, mi], bwd[BLOCK, g, ti, mi] = f, b
                fwd[HEAD, g, ti, mi], bwd[HEAD, g, ti, mi] = f * head_ratio, b * head_ratio
                fwd[EMBED, g, ti, mi], bwd[EMBED, g, ti, mi] = f * 0.02, b * 0.02
            u = 0.3 * type_base[g] / tp
            upd[BLOCK, g, ti] = u
            upd[EMBED, g, ti] = u * float(params[EMBED]) / float(params[BLOCK])
            upd[HEAD, g, ti] = u * float(params[HEAD]) / float(params[BLOCK])

    act_saved = np.zeros((KINDS, n_tp, n_mbs), dtype=np.uint64)
    act_ckpt = np.zeros((KINDS, n_tp, n_mbs), dtype=np.uint64)
    act_work = np.zeros((KINDS, n_tp, n_mbs), dtype=np.uint64)
    p2p = np.zeros(n_mbs, dtype=np.uint64)
    for ti, tp in enumerate(tp_values):
        for mi, mbs in enumerate(mbs_values):
            tok = s * mbs
            act_saved[BLOCK, ti, mi] = _ceil_div(tok * (10 * h * tp + 24 * h + 5 * a * s), tp)
            act_saved[EMBED, ti, mi] = 2 * tok * h
            act_saved[HEAD, ti, mi] = 2 * tok * h + _ceil_div(4 * tok * V, tp)
            for k in range(KINDS):
                act_ckpt[k, ti, mi] = 2 * tok * h
            act_work[BLOCK, ti, mi] = _ceil_div(tok * (8 * h + 2 * a * s), tp)
            act_work[EMBED, ti, mi] = 0
            act_work[HEAD, ti, mi] = _ceil_div(6 * tok * V, tp)
    for mi, mbs in enumerate(mbs_values):
        p2p[mi] = 2 * s * mbs * h

    capacity = np.array([m * GIB for m in type_mem_gib], dtype=np.uint64)
    reserved = np.full(T, GIB, dtype=np.uint64)
    gpn = np.full(T, gpus_per_node, dtype=np.uint32)
    price = np.tile(np.array(type_price, dtype=np.float64), (Z, 1))
    intra_alpha = np.full((Z, T), alpha)
    inter_alpha = np.full((Z, T), alpha)
    intra_inv = np.full((Z, T), _inv_bw(intra_gbs))
    inter_inv = np.full((Z, T), _inv_bw(inter_gbs))
    zone_alpha = np.full((Z, Z), alpha)
    zone_inv = np.zeros((Z, Z))
    egress = np.zeros((Z, Z))
    for z0 in range(Z):
        for z1 in range(z0 + 1, Z):
            bw = zone_bw_fn(rng)
            zone_inv[z0, z1] = zone_inv[z1, z0] = _inv_bw(bw)
            egress[z0, z1] = egress[z1, z0] = egress_usd_per_byte
    avail = np.zeros((Z, T), dtype=np.uint16)
    for z in range(Z):
        for g in range(T):
            avail[z, g] = avail_fn(rng, z, g)

    return Workload(
        name=name, n_blocks=L, has_embed=1, has_head=1, heads=a, gbs=gbs, mul_factor=8,
        dtype_size=2, grad_dtype_size=2, tp_values=list(tp_values), mbs_values=list(mbs_values),
        fwd=fwd, bwd=bwd, upd=upd, params=params, act_saved=act_saved, act_ckpt=act_ckpt,
        act_work=act_work, p2p_bytes=p2p, n_types=T, n_zones=Z, capacity=capacity,
        reserved=reserved, gpus_per_node=gpn, price_per_hour=price, intra_alpha=intra_alpha,
        intra_inv_bw=intra_inv, inter_alpha=inter_alpha, inter_inv_bw=inter_inv,
        zone_alpha=zone_alpha, zone_inv_bw=zone_inv, egress=egress, avail=avail,
        p_values=list(p_values), mbs_idx=list(range(n_mbs)), tp_idx=list(range(n_tp)),
        rc_values=list(rc_values), d_values=list(d_values), seg_max=seg_max,
        objective=objective, budget_factor_over_cheapest=budget_factor)


def with_bandwidth_polynomials(w: Workload, seed: int) -> Workload:
    """Give every link a fitted bandwidth curve that rises with the message size (Sec. 4.1):
    bandwidth(m) = bw * (0.25 + a1 * m + a2 * m^2) with small positive a1, a2 drawn from `seed`,
    bw being the link's constant bandwidth.  The constant-bandwidth fields stay but are ignored."""
    rng = SplitMix64(seed)

    def curve(inv_bw: float):
        bw = 1.0 / inv_bw if inv_bw > 0 else 1e9
        return [0.25 * bw, bw * (2e-8 + 4e-8 * rng.uniform()), bw * 1e-16 * rng.uniform(), 0.0]

    Z, T = w.n_zones, w.n_types
    w.intra_bw_poly = np.array([[curve(w.intra_inv_bw[z, g]) for g in range(T)] for z in range(Z)])
    w.inter_bw_poly = np.array([[curve(w.inter_inv_bw[z, g]) for g in range(T)] for z in range(Z)])
    w.zone_bw_poly = np.array([[curve(w.zone_inv_bw[z0, z1]) for z1 in range(Z)] for z0 in range(Z)])
    w.name += "-bwpoly"
    return w


def _cap_total(avail: np.ndarray, cap: int) -> np.ndarray:
    """Scale counts down proportionally (floor) when their total exceeds `cap`."""
    total = int(avail.sum())
    if total <= cap:
        return avail
    return (avail.astype(np.int64) * cap // total).astype(np.uint16)


SEED_BASE = 0x5A110000


def config1() -> Workload:
    """OPT-350M shape, one zone, 16 x 40 GiB + 16 x 16 GiB GPUs, max throughput (6 768 candidates)."""
    return make_workload(
        "cfg1-opt350m-1zone", seed=SEED_BASE + 1, L=24, h=1024, a=16, s=2048, V=50272, gbs=512,
        type_mem_gib=[40, 16], type_base=[4.3e-4, 4.3e-4 * 2.5], type_price=[2.9, 2.5],
        n_zones=1, gpus_per_node=4, intra_gbs=300.0, inter_gbs=12.5,
        zone_bw_fn=lambda r: 1.0, avail_fn=lambda r, z, g: 16,
        tp_values=[1, 2, 4], mbs_values=[1, 2, 4, 8], p_values=[1, 2, 3, 4, 6, 8, 12, 24],
        d_values=[1, 2, 4, 8, 16, 32], rc_values=[0], objective=OBJ_MAX_THROUGHPUT)


def config2(seed: int = SEED_BASE + 2, name: str = "cfg2-gptneo27b-2zones") -> Workload:
    """GPT-Neo-2.7B shape, 2 zones x 3 types, budget = 1.2 x cheapest feasible (438 984 candidates)."""
    speeds = [1.0, 0.55, 0.25]
    return make_workload(
        name, seed=seed, L=32, h=2560, a=20, s=2048, V=50257, gbs=1024,
        type_mem_gib=[80, 40, 16], type_base=[1.6e-3 / v for v in speeds],
        type_price=[4.0, 2.9, 2.5], n_zones=2, gpus_per_node=4, intra_gbs=300.0, inter_gbs=25.0,
        zone_bw_fn=lambda r: 1.0 + 4.0 * r.uniform(), avail_fn=lambda r, z, g: r.randint(0, 32),
        tp_values=[1, 2, 4], mbs_values=[1, 2, 4, 8], p_values=[1, 2, 4, 8, 16, 32],
        d_values=[1, 2, 4, 8, 16, 32, 64], rc_values=[0], objective=OBJ_MAX_THROUGHPUT,
        budget_factor=1.2)


def config3() -> Workload:
    """OPT-30B shape, 5 zones x 4 types, recomputation flag, max throughput per USD (3.6e8 candidates)."""
    speeds = [1.0, 0.7, 0.55, 0.35]
    w = make_workload(
        "cfg3-opt30b-5zones", seed=SEED_BASE + 3, L=48, h=7168, a=56, s=2048, V=50272, gbs=2048,
        type_mem_gib=[80, 48, 40, 24], type_base=[6.0e-3 / v for v in speeds],
        type_price=[4.0, 3.2, 2.9, 2.6], n_zones=5, gpus_per_node=8, intra_gbs=300.0,
        inter_gbs=25.0, zone_bw_fn=lambda r: r.lognormal(math.log(2.0), 0.7),
        avail_fn=lambda r, z, g: r.poisson(24.0),
        tp_values=[1, 2, 4, 8], mbs_values=[1, 2, 4, 8, 16],
        p_values=[1, 2, 3, 4, 6, 8, 12, 16, 24, 48], d_values=[1, 2, 4, 8, 16, 32, 64, 128],
        rc_values=[0, 1], objective=OBJ_MAX_THROUGHPUT_PER_USD)
    w.avail = _cap_total(w.avail, 512)
    return w


def config4(n_snapshots: int = 200) -> Workload:
    """Workload 2 replayed over availability snapshots: a seeded random walk per (zone, type)."""
    w = config2(name="cfg4-dynamic-availability")
    rng = SplitMix64(SEED_BASE + 4)
    snaps = np.zeros((n_snapshots,) + w.avail.shape, dtype=np.uint16)
    cur = w.avail.astype(np.int64)
    for t in range(n_snapshots):
        snaps[t] = cur.astype(np.uint16)
        for z in range(w.n_zones):
            for g in range(w.n_types):
                step = rng.randint(0, 4) * (1 if rng.next_u64() & 1 else -1)
                cur[z, g] = min(32, max(0, cur[z, g] + step))
    w.snapshots = snaps
    return w


def config5() -> Workload:
    """96-layer stress sweep, 8 zones x 6 types, P up to 16, exhaustive (6.4e9 candidates)."""
    speeds = [1.0, 0.75, 0.45, 0.3, 0.22, 0.15]
    w = make_workload(
        "cfg5-stress-96layer", seed=SEED_BASE + 5, L=96, h=12288, a=96, s=2048, V=50272, gbs=1536,
        type_mem_gib=[192, 141, 80, 48, 40, 24], type_base=[8.0e-3 / v for v in speeds],
        type_price=[9.0, 6.5, 4.0, 3.2, 2.9, 2.6], n_zones=8, gpus_per_node=8, intra_gbs=300.0,
        inter_gbs=25.0, zone_bw_fn=lambda r: r.lognormal(math.log(2.0), 0.7),
        avail_fn=lambda r, z, g: r.poisson(21.0),
        tp_values=[1, 2, 4, 8], mbs_values=[1, 2, 4, 8, 16], p_values=[1, 2, 3, 4, 6, 8, 12, 16],
        d_values=[1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64], rc_values=[0],
        objective=OBJ_MAX_THROUGHPUT)
    w.avail = _cap_total(w.avail, 1024)
    return w


def config6() -> Workload:
    """Shape of the paper's constrained scenario 1 (Sec. 5.2.4): two zones of one region, each with
    128 GPUs of a 40 GiB and of a 16 GiB type; minimise cost per iteration subject to a minimum
    throughput.  GPT-Neo-2.7B-shaped model, global batch 2048 (the paper's evaluation batch size)."""
    w = make_workload(
        "cfg6-min-cost-under-throughput", seed=SEED_BASE + 6, L=32, h=2560, a=20, s=2048, V=50257, gbs=2048,
        type_mem_gib=[40, 16], type_base=[1.6e-3 / 0.55, 1.6e-3 / 0.25], type_price=[2.9, 2.5],
        n_zones=2, gpus_per_node=4, intra_gbs=300.0, inter_gbs=25.0,
        zone_bw_fn=lambda r: 20.0 + 5.0 * r.uniform(), avail_fn=lambda r, z, g: 128,
        tp_values=[1, 2, 4], mbs_values=[1, 2, 4, 8], p_values=[1, 2, 4, 8, 16, 32],
        d_values=[1, 2, 4, 8, 16, 32, 64, 128], rc_values=[0], objective=OBJ_MIN_COST)
    w.min_iters_per_s = 0.2
    return w


def tiny(seed: int = 7, *, n_types: int = 2, n_zones: int = 2, L: int = 4, alpha: float = 2e-5,
         rc_values=(0, 1), objective: int = OBJ_MAX_THROUGHPUT, seg_max: int = 4, p_values=None,
         d_values=(1, 2, 3, 4, 8), tp_values=(1, 2, 4), mbs_values=(1, 2, 4), gbs: int = 32) -> Workload:
    """A cluster small enough to enumerate by brute force; alpha > 0, scarce GPUs, both rc values.
    Up to 8 GPU types and 8 zones (the table limits)."""
    mem = [24, 12, 8, 20, 16, 10, 32, 6][:n_types]
    base = [5.0e-4, 9.0e-4, 1.7e-3, 6.0e-4, 7.5e-4, 1.2e-3, 4.0e-4, 2.2e-3][:n_types]
    price = [3.0, 1.9, 1.1, 2.6, 2.2, 1.5, 3.8, 0.9][:n_types]
    if p_values is None:
        p_values = [p for p in (1, 2, 3, 4) if p <= L]
    return make_workload(
        f"tiny-{seed}", seed=seed, L=L, h=512, a=8, s=512, V=8192, gbs=gbs,
        type_mem_gib=mem, type_base=base, type_price=price, n_zones=n_zones, gpus_per_node=4,
        intra_gbs=100.0, inter_gbs=10.0, zone_bw_fn=lambda r: 0.5 + 2.0 * r.uniform(),
        avail_fn=lambda r, z, g: r.randint(2, 12), tp_values=list(tp_values), mbs_values=list(mbs_values),
        p_values=list(p_values), d_values=list(d_values),
        rc_values=list(rc_values), objective=objective, seg_max=seg_max, alpha=alpha,
        egress_usd_per_byte=2e-11)


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5, 6: config6}


def random_plans(w: Workload, n: int, seed: int, *, max_runs: int = 16, hetero_tp: bool = True):
    """n random explicit plan records as a dict of integer arrays.

    P is drawn from the divisors and non-divisors of the layer count alike, runs have random
    lengths, and each run gets its own (type, zone, tp) when hetero_tp.  Returns
    {"P", "mbs_idx", "rc", "n_runs", "D": [n]; "type", "zone", "tp_idx", "n_stages": [n][16]}.
    """
    rng = SplitMix64(seed)
    out = {k: np.zeros(n, dtype=np.int64) for k in ("P", "mbs_idx", "rc", "n_runs", "D")}
    for k in ("type", "zone", "tp_idx", "n_stages"):
        out[k] = np.zeros((n, 16), dtype=np.int64)
    p_max = min(w.n_blocks, 96)
    for j in range(n):
        P = w.p_values[rng.randint(0, len(w.p_values) - 1)] if rng.uniform() < 0.7 else rng.randint(1, p_max)
        n_runs = rng.randint(1, min(P, max_runs))
        cuts = sorted({rng.randint(1, P - 1) for _ in range(n_runs - 1)}) if P > 1 else []
        bounds = [0] + cuts + [P]
        lens = [bounds[i + 1] - bounds[i] for i in range(len(bounds) - 1)]
        out["P"][j] = P
        out["mbs_idx"][j] = rng.randint(0, len(w.mbs_values) - 1)
        out["rc"][j] = w.rc_values[rng.randint(0, len(w.rc_values) - 1)]
        out["n_runs"][j] = len(lens)
        out["D"][j] = w.d_values[rng.randint(0, len(w.d_values) - 1)]
        tp0 = rng.randint(0, len(w.tp_values) - 1)
        for r, ln in enumerate(lens):
            out["type"][j, r] = rng.randint(0, w.n_types - 1)
            out["zone"][j, r] = rng.randint(0, w.n_zones - 1)
            out["tp_idx"][j, r] = rng.randint(0, len(w.tp_values) - 1) if hetero_tp else tp0
            out["n_stages"][j, r] = ln
    return out


def random_mixed_plans(w: Workload, n: int, seed: int, *, p_max: int = 32, groups_max: int = 4):
    """n random plans whose stages split their D replicas into groups of different (type, tp), as a list of
    dicts {"P", "mbs_idx", "rc", "D", "stages": [{"zone", "groups": [(type, tp_idx, count), ...]}]}.
    About a quarter of the plans have one group in every stage (no mixing)."""
    rng = SplitMix64(seed)
    plans = []
    for _ in range(n):
        P = w.p_values[rng.randint(0, len(w.p_values) - 1)] if rng.uniform() < 0.7 else rng.randint(1, min(w.n_blocks, p_max))
        P = min(P, p_max)
        D = w.d_values[rng.randint(0, len(w.d_values) - 1)]
        plain = rng.uniform() < 0.25
        zone = rng.randint(0, w.n_zones - 1)
        stages = []
        for i in range(P):
            if rng.uniform() < 0.3:
                zone = rng.randint(0, w.n_zones - 1)
            ng = 1 if plain else rng.randint(1, min(groups_max, D))
            cuts = sorted({rng.randint(1, D - 1) for _ in range(ng - 1)}) if D > 1 else []
            bounds = [0] + cuts + [D]
            groups = [(rng.randint(0, w.n_types - 1), rng.randint(0, len(w.tp_values) - 1), bounds[q + 1] - bounds[q])
                      for q in range(len(bounds) - 1)]
            stages.append({"zone": zone, "groups": groups})
        plans.append({"P": P, "mbs_idx": rng.randint(0, len(w.mbs_values) - 1),
                      "rc": w.rc_values[rng.randint(0, len(w.rc_values) - 1)], "D": D, "stages": stages})
    return plans
