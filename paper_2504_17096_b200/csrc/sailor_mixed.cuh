// Simulator for plans whose stages mix GPU types among their D replicas (Sailor Sec. 4.2, Sec. 4.3).
//
// Pipeline k runs on replica k of every stage, replicas being numbered group after group.  Two
// pipelines that use the same group in every stage are identical, so a plan has at most
// 1 + sum_i (groups_i - 1) different pipelines: the replica index is walked from one group boundary
// (of any stage) to the next, and one pipeline is evaluated per interval.  The arithmetic of one
// pipeline is the stage-by-stage evaluation of the plain simulator.
//
// One warp evaluates one plan, lane i owning stage i (a plan has at most 32 stages): the per-stage terms
// of all stages are formed side by side, maxima are taken across the warp, and the sums whose order of
// additions is part of the result (stage times of a pipeline, price rate, transfer cost) are added up in
// stage order from the lanes' terms.  Plans differ widely in depth and in how many pipelines they have;
// a thread per plan kept four lanes of 32 busy on such batches.
#pragma once

#include "sailor_tables.cuh"

namespace sailor {

constexpr uint32_t MIX_FULL = 0xffffffffu;

__device__ __forceinline__ double warp_max_f64(double x) {
#pragma unroll
    for (uint32_t o = 16; o; o >>= 1) x = dmax(x, __shfl_xor_sync(MIX_FULL, x, o));
    return x;
}

__device__ __forceinline__ uint64_t warp_max_u64(uint64_t x) {
#pragma unroll
    for (uint32_t o = 16; o; o >>= 1) {
        const uint64_t y = __shfl_xor_sync(MIX_FULL, (unsigned long long)x, o);
        x = y > x ? y : x;
    }
    return x;
}

// `cnt` points to this warp's per-digit GPU counters (R of them, shared memory).  Every lane of the warp
// calls with the same record and gets the same result.
__device__ inline SimOut simulate_mixed_warp(const TabView& v, const uint16_t* __restrict__ avail,
                                             const sailor_mixed_plan& r, unsigned long long* cnt, uint32_t lane) {
    const TabHdr* h = v.h;
    SimOut o;
    o.t_iter = o.cost = make_nan();
    o.peak_mem = 0;
    o.status = SAILOR_ST_BAD_RECORD;
    const uint32_t P = r.P, D = r.D, mi = r.mbs_idx, rc = r.rc ? 1u : 0u, T = h->T, Z = h->Z, R = h->R;
    if (P < 1 || P > SAILOR_MIX_P_MAX || D < 1 || mi >= h->n_mbs) return o;
    const bool mine = lane < P;

    // this lane's stage
    uint32_t zone = 0, ng = 0, gtype[SAILOR_MIX_GROUPS_MAX], gtpi[SAILOR_MIX_GROUPS_MAX], gcount[SAILOR_MIX_GROUPS_MAX];
#pragma unroll
    for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q) gtype[q] = gtpi[q] = gcount[q] = 0;
    bool bad = false;
    if (mine) {
        const sailor_mixed_stage& s = r.stage[lane];
        zone = s.zone;
        ng = s.n_groups;
        bad = zone >= Z || ng < 1 || ng > SAILOR_MIX_GROUPS_MAX;
#pragma unroll
        for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q)
            if (!bad && q < ng) {
                gtype[q] = s.group[q].type; gtpi[q] = s.group[q].tp_idx; gcount[q] = s.group[q].count;
            }
#pragma unroll
        for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q)
            if (q < ng) bad = bad || gtype[q] >= T || gtpi[q] >= h->n_tp;
    }
    if (__any_sync(MIX_FULL, bad)) return o;

    uint32_t status = 0;
    const uint64_t dm = (uint64_t)D * h->mbs_values[mi];
    if (h->gbs % dm != 0) status |= SAILOR_ST_INVALID;
    const uint64_t n_b = h->gbs / dm;
    const uint32_t base = h->n_blocks / P, extra = h->n_blocks % P;

    // validity, resources, memory per group, update time, synchronisation, price-rate terms: all stages at once
    for (uint32_t d = lane; d < R; d += 32) cnt[d] = 0;
    __syncwarp();
    const double steps = (double)(2 * (uint64_t)(D - 1));
    const double coef = steps / (double)D;
    double sync_l = 0.0, upd_l = 0.0, term[SAILOR_MIX_GROUPS_MAX];
#pragma unroll
    for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q) term[q] = 0.0;
    uint64_t peak_l = 0;
    size_t comp = 0;
    if (mine) {
        const uint32_t i = lane;
        const uint32_t nb = base + (i < extra ? 1u : 0u);
        const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
        const uint64_t inflight = (uint64_t)(P - i) < n_b ? (uint64_t)(P - i) : n_b;
        // what a stage of this make-up needs was formed once per context (per-composition tables)
        comp = (size_t)((e ? 2u : 0u) + (hd ? 1u : 0u)) * h->chain_len + nb;
        uint64_t replicas = 0;
        double gradbytes = 0.0;
#pragma unroll
        for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q)
            if (q < ng) {
                const uint32_t tp = h->tp_values[gtpi[q]];
                replicas += gcount[q];
                if (gcount[q] == 0 || tp > h->gpn[gtype[q]] || h->heads % tp != 0) status |= SAILOR_ST_INVALID;
                atomicAdd(cnt + zone * T + gtype[q], (unsigned long long)gcount[q] * tp);
                const size_t ct = comp * h->n_tp + gtpi[q];
                const uint64_t* mm = v.cmp_mem + ((ct * h->n_mbs + mi) * 2 + rc) * 2;
                const uint64_t m = mm[0] + inflight * mm[1] + h->reserved[gtype[q]];
                if (m > h->capacity[gtype[q]]) status |= SAILOR_ST_OOM;
                peak_l = m > peak_l ? m : peak_l;
                gradbytes = dmax(gradbytes, v.cmp_grad[ct]);      // the ring moves the largest shard (smallest tp)
            }
        if (replicas != D) status |= SAILOR_ST_INVALID;
#pragma unroll
        for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q)
            if (q < ng) {
                const uint32_t d = zone * T + gtype[q], tp = h->tp_values[gtpi[q]];
                upd_l = dmax(upd_l, v.cmp_upd[(comp * T + gtype[q]) * h->n_tp + gtpi[q]]);
                if (D > 1) {
                    const bool intra = ng == 1 && (uint64_t)D * tp <= h->gpn[gtype[q]];
                    sync_l = dmax(sync_l, allreduce_bytes_time(v, d, intra, gradbytes, D, steps, coef));
                }
                term[q] = mul_rn((double)((uint32_t)gcount[q] * tp), v.price_s[d]);
            }
    }
    __syncwarp();                                                // the counters are complete
    if (mine) {
#pragma unroll
        for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q)
            if (q < ng) {
                const uint32_t d = zone * T + gtype[q];
                if (cnt[d] > avail[d]) status |= SAILOR_ST_OVER_AVAIL;
            }
    }
    status = __reduce_or_sync(MIX_FULL, status);
    o.peak_mem = warp_max_u64(peak_l);
    o.status = status;
    if (status & SAILOR_ST_INVALID) return o;
    const double max_sync = warp_max_f64(sync_l), max_u = warp_max_f64(upd_l);
    double rate = 0.0;                                           // stage after stage, group after group
    for (uint32_t i = 0; i < P; ++i) {
        const uint32_t ng_i = __shfl_sync(MIX_FULL, ng, i);
#pragma unroll
        for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q) {
            const double tq = __shfl_sync(MIX_FULL, term[q], i);
            if (q < ng_i) rate = add_rn(rate, tq);
        }
    }

    // the pipelines: from one group boundary to the next all replicas see the same groups
    uint32_t upto[SAILOR_MIX_GROUPS_MAX];                        // replicas up to and including group q of this stage
    {
        uint32_t run = 0;
#pragma unroll
        for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q) { run += gcount[q]; upto[q] = run; }
    }
    const double msg = (double)v.p2p[mi];
    const uint32_t z2 = __shfl_down_sync(MIX_FULL, zone, 1);     // zone of the next stage
    const bool sends = mine && lane + 1 < P;
    double max_pp = 0.0;
    uint32_t k = 0;
    while (k < D) {
        // group of replica k in this lane's stage
        uint32_t g = gtype[0], tpi = gtpi[0], cn = gcount[0], nxt = upto[0];
#pragma unroll
        for (uint32_t q = 1; q < SAILOR_MIX_GROUPS_MAX; ++q)
            if (q < ng && k >= upto[q - 1]) { g = gtype[q]; tpi = gtpi[q]; cn = gcount[q]; nxt = upto[q]; }
        const uint32_t next = __reduce_min_sync(MIX_FULL, mine ? nxt : D);
        const uint32_t g2 = __shfl_down_sync(MIX_FULL, g, 1), tpi2 = __shfl_down_sync(MIX_FULL, tpi, 1),
                       cn2 = __shfl_down_sync(MIX_FULL, cn, 1);
        double t = 0.0;
        if (mine) {
            const double fb = v.cmp_fb[(((comp * T + g) * h->n_tp + tpi) * h->n_mbs + mi) * 2 + rc];
            double c = 0.0;
            if (sends) {
                const uint32_t z = zone;
                if (z != z2) {
                    c = link_time(v.zone_a[z * Z + z2], v.zone_i[z * Z + z2], v.zone_p, z * Z + z2, msg);
                } else if (g == g2 && (uint64_t)cn * h->tp_values[tpi] + (uint64_t)cn2 * h->tp_values[tpi2] <= h->gpn[g]) {
                    const uint32_t d = z * T + g;
                    c = link_time(v.intra_a[d], v.intra_i[d], v.intra_p, d, msg);
                } else {
                    const uint32_t d = z * T + g, d2 = z * T + g2;
                    c = dmax(link_time(v.inter_a[d], v.inter_i[d], v.inter_p, d, msg),
                             link_time(v.inter_a[d2], v.inter_i[d2], v.inter_p, d2, msg));
                }
            }
            t = add_rn(fb, mul_rn(2.0, c));
        }
        const double max_t = warp_max_f64(t);
        double sum_t = 0.0;                                      // in stage order
        for (uint32_t i = 0; i < P; ++i) sum_t = add_rn(sum_t, __shfl_sync(MIX_FULL, t, i));
        max_pp = dmax(max_pp, add_rn(sum_t, mul_rn((double)n_b, max_t)));
        k = next;
    }
    const uint64_t xbytes = 2 * n_b * (uint64_t)D * v.p2p[mi];
    const bool crosses = sends && zone != z2;
    const double cross_cost = crosses ? mul_rn((double)xbytes, v.egress[zone * Z + z2]) : 0.0;
    double c_comm = 0.0;
    for (uint32_t m = __ballot_sync(MIX_FULL, crosses); m; m &= m - 1)        // boundaries in stage order
        c_comm = add_rn(c_comm, __shfl_sync(MIX_FULL, cross_cost, __ffs(m) - 1));
    o.t_iter = add_rn(add_rn(max_pp, max_sync), max_u);
    o.cost = add_rn(mul_rn(rate, o.t_iter), c_comm);
    return o;
}

}  // namespace sailor
