// Plan search kernels: candidates are generated on the device from their flat index,
// simulated (Sailor Sec. 4.3) and reduced to the k best under the objective (Sec. 4.2).
//
// Work decomposition.  A *configuration* is (P, mbs, tp, rc, D); its candidates differ only
// in the (type, zone) digit of each of its nseg segments.  An *item* is one assignment of
// all segments but the last (a prefix); a thread owns one item and walks the last segment's
// digit, so the running sums of the prefix (in stage order, exactly as a stage-by-stage
// evaluation would add them) are formed once and extended per candidate.  A *chunk* is
// PLAN_THREADS consecutive items of one configuration; blocks take chunks from an atomic
// counter, and rebuild the per-configuration stage tables in shared memory only when the
// configuration changes.  Lanes of a warp hold consecutive prefixes of one configuration,
// so loop trip counts are warp-uniform and per-digit table reads are broadcasts.
#pragma once

#include "sailor_tables.cuh"

namespace sailor {

constexpr int PLAN_THREADS = 256;
constexpr int PLAN_WARPS = PLAN_THREADS / 32;
constexpr unsigned FULL = 0xffffffffu;
constexpr uint32_t WAIT_LIMIT = 1u << 22;   // bound of every spin-wait in this file

struct Hit {
    double score;
    uint64_t flat;
};

struct Ctrl {                       // one per context, device memory
    unsigned int work_counter;      // next chunk to hand out (cleared per pass)
    unsigned int n_found;
    unsigned long long stats[6];    // total, invalid, oom, over_avail, over_constraint, feasible
    unsigned long long min_cost_bits;   // min C_iter over feasible candidates, as ordered bits
    double budget;                  // written by the cheapest-plan pass for the next pass
    unsigned int error;             // non-zero: a kernel gave up (bounded wait ran out); sticky
    unsigned int _pad;
};

struct PlanParams {
    const unsigned char* blob;
    const uint16_t* avail;
    const uint32_t* cfg_chunk_start;   // [n_config + 1]
    const uint64_t* cfg_flat_base;     // [n_config]
    Ctrl* ctrl;
    Hit* partial;                      // [grid][SAILOR_K_MAX]
    uint32_t* partial_n;               // [grid]
    SpaceDesc sp;
    uint32_t n_config;
    uint32_t chunk_lo, chunk_hi, batch;
    uint64_t flat_lo, flat_hi;
    uint32_t k;
    uint32_t eval_all;
    uint32_t budget_from_ctrl;         // read the budget from ctrl->budget
    uint32_t p_max;                    // largest P of the space (sizes the stage tables)
    double budget;                     // <= 0: none
    double min_rate;                   // <= 0: none
};

// ---- bounded bulk copy global -> shared (non-multicast cp.async.bulk + mbarrier) ------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Copies `bytes` (multiple of 16, both addresses 16-byte aligned) with one bulk-copy
// instruction issued by thread 0 and waits for it with a bounded spin.  Returns false if the
// wait ran out; the caller then falls back to plain loads and raises the error flag.
__device__ __forceinline__ bool bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* mbar) {
    const uint32_t bar = smem_u32(mbar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(bar)
                     : "memory");
    }
    uint32_t done = 0;
    for (uint32_t it = 0; it < WAIT_LIMIT && !done; ++it) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar)
            : "memory");
    }
    return __syncthreads_and((int)done) != 0;
}

// ---- warp-resident sorted top-k list: lane j holds the j-th best (score, flat) -------------
struct WarpTopK {
    double score;      // this lane's element
    uint64_t flat;
    double thr_score;  // element k-1 (warp-uniform): only strictly better candidates enter
    uint64_t thr_flat;

    __device__ __forceinline__ void init() {
        score = thr_score = make_inf();
        flat = thr_flat = ~0ull;
    }
    // Insert one candidate known to every lane.  (score, flat) pairs are unique.
    __device__ __forceinline__ void insert(double s, uint64_t f, uint32_t k, uint32_t lane) {
        if (!(s < thr_score || (s == thr_score && f < thr_flat))) return;   // warp-uniform
        const bool before = (score < s) || (score == s && flat < f);
        const uint32_t pos = __popc(__ballot_sync(FULL, before));           // sorted: a prefix of lanes
        const double ps = __shfl_up_sync(FULL, score, 1);
        const uint64_t pf = __shfl_up_sync(FULL, flat, 1);
        if (lane > pos) { score = ps; flat = pf; }
        else if (lane == pos) { score = s; flat = f; }
        thr_score = __shfl_sync(FULL, score, k - 1);
        thr_flat = __shfl_sync(FULL, flat, k - 1);
    }
    // Offer per-lane candidates: `want` marks lanes whose candidate may qualify.
    __device__ __forceinline__ void offer(bool want, double s, uint64_t f, uint32_t k, uint32_t lane) {
        unsigned m = __ballot_sync(FULL, want);
        while (m) {
            const int src = __ffs(m) - 1;
            m &= m - 1;
            insert(__shfl_sync(FULL, s, src), __shfl_sync(FULL, f, src), k, lane);
        }
    }
};

// ---- per-configuration tables in shared memory ---------------------------------------------
struct CfgShared {
    // scalars (written by thread 0 / the build, read by all)
    Config cfg;
    uint32_t valid;              // gbs % (D*mbs) == 0 and heads % tp == 0
    uint32_t seg_a[SAILOR_SEG_MAX + 1];   // first stage of each segment; seg_a[nseg] = P
    uint32_t need[SAILOR_SEG_MAX];        // GPUs a segment takes of its digit: D * tp * stages
    uint64_t n_b;
    uint64_t n_items;            // R^(nseg-1)
    uint64_t invalid_mask;       // digit d: tp > gpus_per_node[type(d)]
    uint64_t oom_mask[SAILOR_SEG_MAX];    // digit d: some stage of the segment does not fit type(d)
    uint64_t avail_last;         // digit d: need[last] <= avail[d]
    uint32_t cur_config;
    uint32_t next_chunk;
    uint32_t oom_stage[SAILOR_P_MAX];     // per stage: bit g set when the stage does not fit type g
    uint64_t params[SAILOR_P_MAX];
    unsigned long long stat[6];
    uint64_t mbar;
};

struct CfgArrays {               // pointers into dynamic shared memory
    double *fb, *uu;             // [P][T]   f+b (+f if rc), update
    double* tself;               // [P][R]   t_i when stage i+1 has the same digit (last stage: no message)
    double *seg_tmax, *seg_sync, *seg_upd;   // [nseg][R]
    double* rate_d;              // [R]      D * tp * price per second
    double* c2x;                 // [R][R]   2 * message time, index [next digit][this digit]
    double* commx;               // [Z][Z]   transfer cost of one boundary, index [next zone][this zone]
    uint32_t* availv;            // [R]
};

__host__ __device__ inline size_t plan_smem_bytes(uint32_t static_bytes, uint32_t p_max, uint32_t T, uint32_t Z) {
    const size_t R = (size_t)T * Z;
    size_t n = static_bytes;
    n += sizeof(double) * (2 * (size_t)p_max * T + (size_t)p_max * R + 3 * SAILOR_SEG_MAX * R + R + R * R + (size_t)Z * Z);
    n += sizeof(uint32_t) * R;
    return (n + 15) & ~(size_t)15;
}

__device__ __forceinline__ void carve(unsigned char* dyn, uint32_t static_bytes, uint32_t p_max, uint32_t T,
                                      uint32_t Z, CfgArrays& a) {
    const uint32_t R = T * Z;
    double* p = reinterpret_cast<double*>(dyn + static_bytes);
    a.fb = p;        p += (size_t)p_max * T;
    a.uu = p;        p += (size_t)p_max * T;
    a.tself = p;     p += (size_t)p_max * R;
    a.seg_tmax = p;  p += SAILOR_SEG_MAX * R;
    a.seg_sync = p;  p += SAILOR_SEG_MAX * R;
    a.seg_upd = p;   p += SAILOR_SEG_MAX * R;
    a.rate_d = p;    p += R;
    a.c2x = p;       p += (size_t)R * R;
    a.commx = p;     p += (size_t)Z * Z;
    a.availv = reinterpret_cast<uint32_t*>(p);
}

// Build the tables of configuration `c`.  Called by the whole block; ends synchronised.
__device__ void build_config(const PlanParams& pp, const TabView& v, CfgShared& cs, CfgArrays& a, uint32_t c) {
    const TabHdr* h = v.h;
    const uint32_t T = h->T, Z = h->Z, R = h->R, tid = threadIdx.x;
    if (tid == 0) {
        Config k = config_of(pp.sp, c);
        cs.cfg = k;
        const uint32_t tp = h->tp_values[k.tpi];
        const uint64_t dm = (uint64_t)k.D * h->mbs_values[k.mi];
        cs.valid = (k.D >= 1 && h->gbs % dm == 0 && h->heads % tp == 0) ? 1u : 0u;
        cs.n_b = k.D >= 1 ? h->gbs / dm : 0;
        for (uint32_t s = 0; s <= k.nseg; ++s) cs.seg_a[s] = (s * k.P + k.nseg - 1) / k.nseg;
        for (uint32_t s = 0; s < k.nseg; ++s) {
            cs.need[s] = k.D * tp * (cs.seg_a[s + 1] - cs.seg_a[s]);
            cs.oom_mask[s] = 0;
        }
        cs.n_items = ipow64(R, k.nseg - 1);
        uint64_t inv = 0;
        for (uint32_t d = 0; d < R; ++d)
            if (tp > h->gpn[d % T]) inv |= 1ull << d;
        cs.invalid_mask = inv;
        cs.cur_config = c;
    }
    for (uint32_t i = tid; i < SAILOR_P_MAX; i += PLAN_THREADS) cs.oom_stage[i] = 0;
    __syncthreads();
    const Config k = cs.cfg;
    const uint32_t P = k.P, tp = h->tp_values[k.tpi];
    if (!cs.valid) return;             // nothing of this configuration is evaluated (block-uniform)

    // phase A: per (stage, type) times and memory
    const uint32_t base = h->n_blocks / P, extra = h->n_blocks % P;
    for (uint32_t x = tid; x < P * T; x += PLAN_THREADS) {
        const uint32_t i = x / T, g = x % T;
        const uint32_t nb = base + (i < extra ? 1u : 0u);
        const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
        const StageTimes st = stage_times(v, g, k.tpi, k.mi, nb, e, hd);
        const double b = k.rc ? add_rn(st.b, st.f) : st.b;
        a.fb[x] = add_rn(st.f, b);
        a.uu[x] = st.u;
        const uint64_t inflight = (uint64_t)(P - i) < cs.n_b ? (uint64_t)(P - i) : cs.n_b;
        const StageMem sm = stage_memory(v, k.tpi, k.mi, k.rc, nb, e, hd, inflight);
        if (sm.mem + h->reserved[g] > h->capacity[g]) atomicOr(&cs.oom_stage[i], 1u << g);
        if (g == 0) cs.params[i] = sm.params;
    }
    for (uint32_t d = tid; d < R; d += PLAN_THREADS) {
        a.availv[d] = pp.avail[d];
        a.rate_d[d] = mul_rn((double)(k.D * tp), v.price_s[d]);
    }
    __syncthreads();

    // phase B: t_i with the next stage on the same digit; boundary tables
    const double msg = (double)v.p2p[k.mi];
    for (uint32_t x = tid; x < P * R; x += PLAN_THREADS) {
        const uint32_t i = x / R, d = x % R, g = d % T, z = d / T;
        double t = a.fb[i * T + g];
        if (i + 1 < P) t = add_rn(t, mul_rn(2.0, boundary_time(v, g, z, tp, g, z, tp, k.D, msg)));
        a.tself[x] = t;
    }
    const uint64_t xbytes = 2 * cs.n_b * (uint64_t)k.D * v.p2p[k.mi];
    for (uint32_t x = tid; x < R * R; x += PLAN_THREADS) {
        const uint32_t dn = x / R, d = x % R;      // [next][this]
        a.c2x[x] = mul_rn(2.0, boundary_time(v, d % T, d / T, tp, dn % T, dn / T, tp, k.D, msg));
    }
    for (uint32_t x = tid; x < Z * Z; x += PLAN_THREADS) {
        const uint32_t zn = x / Z, z = x % Z;      // [next][this]
        a.commx[x] = (z != zn) ? mul_rn((double)xbytes, v.egress[z * Z + zn]) : 0.0;
    }
    __syncthreads();
    // phase C: per (segment, digit) maxima and memory masks
    for (uint32_t x = tid; x < k.nseg * R; x += PLAN_THREADS) {
        const uint32_t s = x / R, d = x % R, g = d % T, z = d / T;
        const uint32_t sa = cs.seg_a[s], se = cs.seg_a[s + 1];
        // the last stage of a non-final segment talks to the next segment: its t is not in tself
        const uint32_t t_end = (s + 1 < k.nseg) ? se - 1 : se;
        double tm = 0.0, sy = 0.0, up = 0.0;
        bool oom = false;
        for (uint32_t i = sa; i < se; ++i) {
            if (i < t_end) tm = dmax(tm, a.tself[i * R + d]);
            sy = dmax(sy, sync_time(v, g, z, tp, k.D, cs.params[i]));
            up = dmax(up, a.uu[i * T + g]);
            oom |= (cs.oom_stage[i] >> g) & 1u;
        }
        a.seg_tmax[x] = tm;
        a.seg_sync[x] = sy;
        a.seg_upd[x] = up;
        if (oom) atomicOr(reinterpret_cast<unsigned long long*>(&cs.oom_mask[s]), 1ull << d);
    }
    if (tid == 0) {
        uint64_t m = 0;
        for (uint32_t d = 0; d < R; ++d)
            if (cs.need[k.nseg - 1] <= a.availv[d]) m |= 1ull << d;
        cs.avail_last = m;
    }
    __syncthreads();
}

__device__ __forceinline__ uint64_t warp_or64(uint64_t x) {
    const uint32_t lo = __reduce_or_sync(FULL, (uint32_t)x);
    const uint32_t hi = __reduce_or_sync(FULL, (uint32_t)(x >> 32));
    return ((uint64_t)hi << 32) | lo;
}

struct Counters {
    uint32_t invalid, oom, over_avail, over_constr, feasible, total;
    double min_cost;
};

// Add a warp's per-thread counters to the block's 64-bit sums and clear them.
__device__ __forceinline__ void flush_counters(CfgShared& cs, Counters& cnt, uint32_t lane) {
    uint32_t* vals[6] = {&cnt.total, &cnt.invalid, &cnt.oom, &cnt.over_avail, &cnt.over_constr, &cnt.feasible};
#pragma unroll
    for (int j = 0; j < 6; ++j) {
        unsigned long long s = *vals[j];
#pragma unroll
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
        if (lane == 0 && s) atomicAdd(&cs.stat[j], s);
        *vals[j] = 0;
    }
}

// One item per lane: fixed prefix digits, walk the last segment's digit.
template <int NSEG, int OBJ, bool CONSTR>
__device__ __forceinline__ void run_items(const PlanParams& pp, const CfgShared& cs, const CfgArrays& a,
                                          uint32_t T, uint32_t Z, uint32_t R, uint64_t q, bool active,
                                          uint64_t item_flat, double budget, WarpTopK& top, Counters& cnt,
                                          uint32_t lane) {
    constexpr uint32_t last = NSEG - 1;
    // ---- prefix: segments 0 .. NSEG-2 --------------------------------------------------------
    uint32_t dg[NSEG > 1 ? NSEG - 1 : 1];
    {
        uint64_t x = active ? q : 0;
#pragma unroll
        for (int s = NSEG - 2; s >= 0; --s) { dg[s] = (uint32_t)(x % R); x /= R; }
    }
    double acc = 0.0, mx = 0.0, sy = 0.0, up = 0.0, rate = 0.0, cc = 0.0;
    bool p_inv = false, p_oom = false, p_over = false;
#pragma unroll
    for (int s = 0; s < NSEG - 1; ++s) {
        const uint32_t d = dg[s];
        const uint32_t sa = cs.seg_a[s], se = cs.seg_a[s + 1];
        const double rd = a.rate_d[d];
        for (uint32_t i = sa; i + 1 < se; ++i) {          // stages followed by the same digit
            acc = add_rn(acc, a.tself[i * R + d]);
            rate = add_rn(rate, rd);
        }
        mx = dmax(mx, a.seg_tmax[s * R + d]);
        sy = dmax(sy, a.seg_sync[s * R + d]);
        up = dmax(up, a.seg_upd[s * R + d]);
        rate = add_rn(rate, rd);                          // the segment's last stage
        if (s < NSEG - 2) {                               // its message goes to the next prefix digit
            const uint32_t dn = dg[s + 1];
            const double tb = add_rn(a.fb[(se - 1) * T + d % T], a.c2x[dn * R + d]);
            acc = add_rn(acc, tb);
            mx = dmax(mx, tb);
            cc = add_rn(cc, a.commx[(dn / T) * Z + d / T]);
        }
        p_inv |= (cs.invalid_mask >> d) & 1;
        p_oom |= (cs.oom_mask[s] >> d) & 1;
        uint32_t tot = 0;                                 // demand of this digit over the prefix
#pragma unroll
        for (int s2 = 0; s2 < NSEG - 1; ++s2) tot += (dg[s2] == d) ? cs.need[s2] : 0u;
        p_over |= tot > a.availv[d];
    }
    // ---- which last digits are in range / valid / fit / available ------------------------------
    uint64_t range = R == 64 ? ~0ull : ((1ull << R) - 1);
    if (item_flat < pp.flat_lo) {
        const uint64_t skip = pp.flat_lo - item_flat;
        range = skip >= 64 ? 0 : range & (~0ull << skip);
    }
    if (item_flat + R > pp.flat_hi) {
        const uint64_t keep = pp.flat_hi > item_flat ? pp.flat_hi - item_flat : 0;
        range = keep >= 64 ? range : range & ((1ull << keep) - 1);
    }
    if (!active) range = 0;
    const uint64_t valid_l = range & ~cs.invalid_mask;
    const uint64_t good_l = valid_l & ~cs.oom_mask[last];
    uint64_t ok = good_l & cs.avail_last;
#pragma unroll
    for (int s = 0; s < NSEG - 1; ++s) {                  // a last digit equal to a prefix digit adds up
        const uint32_t d = dg[s];
        uint32_t tot = cs.need[last];
#pragma unroll
        for (int s2 = 0; s2 < NSEG - 1; ++s2) tot += (dg[s2] == d) ? cs.need[s2] : 0u;
        if (tot > a.availv[d]) ok &= ~(1ull << d);
    }
    // exactly one class per candidate: invalid, then oom, then over availability
    const uint32_t n_range = __popcll(range);
    cnt.total += n_range;
    if (p_inv) { cnt.invalid += n_range; ok = 0; }
    else {
        cnt.invalid += n_range - __popcll(valid_l);
        if (p_oom) { cnt.oom += __popcll(valid_l); ok = 0; }
        else {
            cnt.oom += __popcll(valid_l) - __popcll(good_l);
            if (p_over) { cnt.over_avail += __popcll(good_l); ok = 0; }
            else cnt.over_avail += __popcll(good_l) - __popcll(ok);
        }
    }
    const uint32_t n_ok = __popcll(ok);
    if (!CONSTR) cnt.feasible += n_ok;

    // ---- the candidates -----------------------------------------------------------------------
    uint64_t walk = pp.eval_all ? warp_or64(range) : warp_or64(ok);   // warp-uniform: skip dead digits
    const uint32_t la = cs.seg_a[last], le = cs.seg_a[last + 1];
    const double nb = (double)cs.n_b;
    double fb_b = 0.0;
    uint32_t d_prev = 0, z_prev = 0;
    if (NSEG > 1) {
        d_prev = dg[NSEG > 1 ? NSEG - 2 : 0];
        z_prev = d_prev / T;
        fb_b = a.fb[(la - 1) * T + d_prev % T];
    }
    uint32_t feas = 0;
    while (walk) {
        const uint32_t d = __ffsll((long long)walk) - 1;
        walk &= walk - 1;
        double t_sum = acc, t_max = mx;
        double c_comm = cc;
        if (NSEG > 1) {                                   // last stage of the prefix sends to digit d
            const double tb = add_rn(fb_b, a.c2x[d * R + d_prev]);
            t_sum = add_rn(t_sum, tb);
            t_max = dmax(t_max, tb);
            c_comm = add_rn(c_comm, a.commx[(d / T) * Z + z_prev]);
        }
        double r = rate;
        const double rd = a.rate_d[d];
        for (uint32_t i = la; i < le; ++i) {
            t_sum = add_rn(t_sum, a.tself[i * R + d]);
            r = add_rn(r, rd);
        }
        t_max = dmax(t_max, a.seg_tmax[last * R + d]);
        const double t_pp = add_rn(t_sum, mul_rn(nb, t_max));
        const double t_iter = add_rn(add_rn(t_pp, dmax(sy, a.seg_sync[last * R + d])), dmax(up, a.seg_upd[last * R + d]));
        const double cost = add_rn(mul_rn(r, t_iter), c_comm);
        bool good = (ok >> d) & 1;
        if (CONSTR) {
            if (budget > 0.0) good &= !(cost > budget);
            if (pp.min_rate > 0.0) good &= !(1.0 / t_iter < pp.min_rate);
            feas += good;
        }
        const double score = OBJ == SAILOR_OBJ_MAX_THROUGHPUT ? t_iter
                           : OBJ == SAILOR_OBJ_MIN_COST ? cost : mul_rn(t_iter, cost);
        if (good && cost < cnt.min_cost) cnt.min_cost = cost;
        const bool want = good && score <= top.thr_score;
        if (__any_sync(FULL, want)) top.offer(want, score, item_flat + d, pp.k, lane);
    }
    if (CONSTR) {
        cnt.feasible += feas;
        cnt.over_constr += n_ok - feas;
    }
}

template <int OBJ, bool CONSTR>
__global__ void __launch_bounds__(PLAN_THREADS) plan_kernel(const __grid_constant__ PlanParams pp) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ CfgShared cs;
    __shared__ Hit s_hits[PLAN_WARPS][SAILOR_K_MAX];

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TabHdr* gh = reinterpret_cast<const TabHdr*>(pp.blob);
    const uint32_t static_bytes = gh->static_bytes;

    // stage the static tables: one bulk copy, bounded wait, plain-load fallback
    if (!bulk_load(dyn, pp.blob, static_bytes, &cs.mbar)) {
        if (tid == 0) atomicExch(&pp.ctrl->error, 1u);
        for (uint32_t x = tid; x < static_bytes / 16; x += PLAN_THREADS)
            reinterpret_cast<uint4*>(dyn)[x] = reinterpret_cast<const uint4*>(pp.blob)[x];
        __syncthreads();
    }
    TabView v;
    v.bind(dyn, pp.blob);
    const uint32_t T = v.h->T, Z = v.h->Z, R = v.h->R;
    CfgArrays a;
    carve(dyn, static_bytes, pp.p_max, T, Z, a);

    if (tid == 0) cs.cur_config = 0xffffffffu;
    if (tid < 6) cs.stat[tid] = 0;
    WarpTopK top;
    top.init();
    Counters cnt = {0, 0, 0, 0, 0, 0, make_inf()};
    const double budget = pp.budget_from_ctrl ? pp.ctrl->budget : pp.budget;
    __syncthreads();

    uint32_t c = 0;     // configuration of the current chunk (monotone within a batch)
    for (;;) {
        if (tid == 0) cs.next_chunk = pp.chunk_lo + atomicAdd(&pp.ctrl->work_counter, pp.batch);
        __syncthreads();
        const uint32_t first = cs.next_chunk;
        if (first >= pp.chunk_hi) break;
        const uint32_t end = min(first + pp.batch, pp.chunk_hi);
        {   // configuration of the first chunk: binary search (uniform)
            uint32_t lo = 0, hi = pp.n_config;
            while (hi - lo > 1) {
                const uint32_t mid = (lo + hi) >> 1;
                if (pp.cfg_chunk_start[mid] <= first) lo = mid; else hi = mid;
            }
            c = lo;
        }
        for (uint32_t ch = first; ch < end; ++ch) {
            while (ch >= pp.cfg_chunk_start[c + 1]) ++c;
            if (cs.cur_config != c) {
                __syncthreads();
                build_config(pp, v, cs, a, c);
            }
            const uint64_t q = (uint64_t)(ch - pp.cfg_chunk_start[c]) * PLAN_THREADS + tid;
            const bool active = q < cs.n_items;
            const uint64_t item_flat = pp.cfg_flat_base[c] + q * R;
            if (!cs.valid) {
                // every candidate of the configuration is invalid; count those in range
                if (active) {
                    const uint64_t lo = item_flat > pp.flat_lo ? item_flat : pp.flat_lo;
                    const uint64_t hi = item_flat + R < pp.flat_hi ? item_flat + R : pp.flat_hi;
                    const uint32_t n = hi > lo ? (uint32_t)(hi - lo) : 0u;
                    cnt.total += n;
                    cnt.invalid += n;
                }
                continue;
            }
            switch (cs.cfg.nseg) {
                case 1: run_items<1, OBJ, CONSTR>(pp, cs, a, T, Z, R, q, active, item_flat, budget, top, cnt, lane); break;
                case 2: run_items<2, OBJ, CONSTR>(pp, cs, a, T, Z, R, q, active, item_flat, budget, top, cnt, lane); break;
                case 3: run_items<3, OBJ, CONSTR>(pp, cs, a, T, Z, R, q, active, item_flat, budget, top, cnt, lane); break;
                default: run_items<4, OBJ, CONSTR>(pp, cs, a, T, Z, R, q, active, item_flat, budget, top, cnt, lane); break;
            }
        }
        // per-thread counters are 32 bits wide: hand them to the block's 64-bit sums in time
        if (__any_sync(FULL, cnt.total > (1u << 30))) flush_counters(cs, cnt, lane);
        __syncthreads();     // next_chunk and the tables are reused
    }

    // ---- block reduction: counters, then the warps' lists ---------------------------------------
    flush_counters(cs, cnt, lane);
    {
        unsigned long long mc = (unsigned long long)__double_as_longlong(cnt.min_cost);   // positive: bits order
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(FULL, mc, o);
            mc = other < mc ? other : mc;
        }
        if (lane == 0) atomicMin(&pp.ctrl->min_cost_bits, mc);
    }
    s_hits[warp][lane].score = top.score;
    s_hits[warp][lane].flat = top.flat;
    __syncthreads();
    if (tid < 6 && cs.stat[tid]) atomicAdd(&pp.ctrl->stats[tid], cs.stat[tid]);
    if (warp == 0) {
        for (uint32_t w = 1; w < PLAN_WARPS; ++w)
            for (uint32_t j = 0; j < pp.k; ++j) {
                const Hit hj = s_hits[w][j];
                if (hj.flat == ~0ull) break;             // lists are sorted; the rest is empty
                top.insert(hj.score, hj.flat, pp.k, lane);
            }
        const uint32_t n = __popc(__ballot_sync(FULL, top.flat != ~0ull && lane < pp.k));
        if (lane < pp.k) {
            pp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].score = top.score;
            pp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].flat = top.flat;
        }
        if (lane == 0) pp.partial_n[blockIdx.x] = n;
    }
}

// Merge the blocks' lists, then simulate the winners in full for the result records.
struct MergeParams {
    const unsigned char* blob;
    const uint16_t* avail;
    const Hit* partial;
    const uint32_t* partial_n;
    Ctrl* ctrl;
    sailor_result* results;            // [k] device
    SpaceDesc sp;
    uint32_t n_partial, k, obj;
    double budget_factor;              // > 0: write ctrl->budget = factor * best cost for the next pass
};

constexpr int MERGE_THREADS = 256;

__global__ void __launch_bounds__(MERGE_THREADS) merge_kernel(const __grid_constant__ MergeParams mp) {
    __shared__ Hit s_hits[MERGE_THREADS / 32][SAILOR_K_MAX];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = MERGE_THREADS / 32;
    WarpTopK top;
    top.init();
    for (uint32_t b = warp; b < mp.n_partial; b += nw) {
        const uint32_t n = mp.partial_n[b];
        for (uint32_t j = 0; j < n; ++j) {
            const Hit hj = mp.partial[(size_t)b * SAILOR_K_MAX + j];
            top.insert(hj.score, hj.flat, mp.k, lane);
        }
    }
    s_hits[warp][lane].score = top.score;
    s_hits[warp][lane].flat = top.flat;
    __syncthreads();
    if (warp != 0) return;
    for (uint32_t w = 1; w < nw; ++w)
        for (uint32_t j = 0; j < mp.k; ++j) {
            const Hit hj = s_hits[w][j];
            if (hj.flat == ~0ull) break;
            top.insert(hj.score, hj.flat, mp.k, lane);
        }
    const bool have = lane < mp.k && top.flat != ~0ull;
    const uint32_t n = __popc(__ballot_sync(FULL, have));
    TabView v;
    v.bind(mp.blob, mp.blob);
    double best_cost = 0.0;
    if (have) {
        sailor_result r;
        r.flat = top.flat;
        r.score = top.score;
        r._pad = 0;
        decode_flat(mp.sp, v.h->T, v.h->Z, top.flat, &r.plan);
        const SimOut o = simulate_record(v, mp.avail, r.plan);
        r.t_iter = o.t_iter;
        r.cost = o.cost;
        r.peak_mem = o.peak_mem;
        r.status = o.status;
        mp.results[lane] = r;
        best_cost = o.cost;
    }
    best_cost = __shfl_sync(FULL, best_cost, 0);
    if (lane == 0) {
        mp.ctrl->n_found = n;
        if (mp.budget_factor > 0.0)
            mp.ctrl->budget = n ? mul_rn(mp.budget_factor, best_cost) : make_inf();
    }
}

}  // namespace sailor
