// Simulator for plans whose stages mix GPU types among their D replicas (Sailor Sec. 4.2, Sec. 4.3).
//
// Pipeline k runs on replica k of every stage, replicas being numbered group after group.  Two
// pipelines that use the same group in every stage are identical, so a plan has at most
// 1 + sum_i (groups_i - 1) different pipelines: the replica index is walked from one group boundary
// (of any stage) to the next, and one pipeline is evaluated per interval.  The arithmetic of one
// pipeline is the stage-by-stage evaluation of the plain simulator.
#pragma once

#include "sailor_tables.cuh"

namespace sailor {

// `cnt` points to this thread's per-digit GPU counters (digit d at cnt[d * cnt_stride]).
__device__ inline SimOut simulate_mixed_record(const TabView& v, const uint16_t* __restrict__ avail,
                                               const sailor_mixed_plan& r, uint32_t* cnt, uint32_t cnt_stride) {
    const TabHdr* h = v.h;
    SimOut o;
    o.t_iter = o.cost = make_nan();
    o.peak_mem = 0;
    o.status = SAILOR_ST_BAD_RECORD;
    const uint32_t P = r.P, D = r.D, mi = r.mbs_idx, rc = r.rc ? 1u : 0u, T = h->T, Z = h->Z;
    if (P < 1 || P > SAILOR_MIX_P_MAX || D < 1 || mi >= h->n_mbs) return o;
    for (uint32_t i = 0; i < P; ++i) {
        const sailor_mixed_stage& s = r.stage[i];
        if (s.zone >= Z || s.n_groups < 1 || s.n_groups > SAILOR_MIX_GROUPS_MAX) return o;
        for (uint32_t q = 0; q < s.n_groups; ++q)
            if (s.group[q].type >= T || s.group[q].tp_idx >= h->n_tp) return o;
    }
    uint32_t status = 0;
    const uint64_t dm = (uint64_t)D * h->mbs_values[mi];
    if (h->gbs % dm != 0) status |= SAILOR_ST_INVALID;
    const uint64_t n_b = h->gbs / dm;
    const uint32_t base = h->n_blocks / P, extra = h->n_blocks % P;

    // validity, resources (saturating), memory per group, update time, synchronisation, price rate
    for (uint32_t d = 0; d < h->R; ++d) cnt[d * cnt_stride] = 0;
    const double steps = (double)(2 * (uint64_t)(D - 1));
    const double coef = steps / (double)D;
    double max_sync = 0.0, max_u = 0.0, rate = 0.0;
    uint64_t peak = 0;
    for (uint32_t i = 0; i < P; ++i) {
        const sailor_mixed_stage& s = r.stage[i];
        const uint32_t nb = base + (i < extra ? 1u : 0u), ng = s.n_groups;
        const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
        const uint64_t inflight = (uint64_t)(P - i) < n_b ? (uint64_t)(P - i) : n_b;
        // what a stage of this make-up needs was formed once per context (per-composition tables)
        const size_t comp = (size_t)((e ? 2u : 0u) + (hd ? 1u : 0u)) * h->chain_len + nb;
        uint64_t replicas = 0;
        double gradbytes = 0.0;
        for (uint32_t q = 0; q < ng; ++q) {
            const sailor_replica_group gr = s.group[q];
            const uint32_t tp = h->tp_values[gr.tp_idx];
            replicas += gr.count;
            if (gr.count == 0 || tp > h->gpn[gr.type] || h->heads % tp != 0) status |= SAILOR_ST_INVALID;
            uint32_t* c = cnt + (s.zone * T + gr.type) * cnt_stride;
            const uint64_t sum = (uint64_t)*c + (uint64_t)gr.count * tp;
            *c = sum > 0xffffffffull ? 0xffffffffu : (uint32_t)sum;
            const size_t ct = comp * h->n_tp + gr.tp_idx;
            const uint64_t* mm = v.cmp_mem + ((ct * h->n_mbs + mi) * 2 + rc) * 2;
            const uint64_t m = mm[0] + inflight * mm[1] + h->reserved[gr.type];
            if (m > h->capacity[gr.type]) status |= SAILOR_ST_OOM;
            peak = m > peak ? m : peak;
            gradbytes = dmax(gradbytes, v.cmp_grad[ct]);          // the ring moves the largest shard (smallest tp)
        }
        if (replicas != D) status |= SAILOR_ST_INVALID;
        double sync = 0.0;
        for (uint32_t q = 0; q < ng; ++q) {
            const sailor_replica_group gr = s.group[q];
            const uint32_t d = s.zone * T + gr.type, tp = h->tp_values[gr.tp_idx];
            max_u = dmax(max_u, v.cmp_upd[(comp * T + gr.type) * h->n_tp + gr.tp_idx]);
            if (D > 1) {
                const bool intra = ng == 1 && (uint64_t)D * tp <= h->gpn[gr.type];
                sync = dmax(sync, allreduce_bytes_time(v, d, intra, gradbytes, D, steps, coef));
            }
            rate = add_rn(rate, mul_rn((double)((uint32_t)gr.count * tp), v.price_s[d]));
        }
        max_sync = dmax(max_sync, sync);
    }
    for (uint32_t i = 0; i < P; ++i)
        for (uint32_t q = 0; q < r.stage[i].n_groups; ++q) {
            const uint32_t d = r.stage[i].zone * T + r.stage[i].group[q].type;
            if (cnt[d * cnt_stride] > avail[d]) status |= SAILOR_ST_OVER_AVAIL;
        }
    o.peak_mem = peak;
    o.status = status;
    if (status & SAILOR_ST_INVALID) return o;

    // the pipelines: from one group boundary to the next all replicas see the same groups
    const double msg = (double)v.p2p[mi];
    double max_pp = 0.0;
    uint32_t k = 0;
    while (k < D) {
        uint32_t next = D;
        double sum_t = 0.0, max_t = 0.0;
        // group of replica k in stage 0; the loop carries the group of stage i into the step for stage i + 1
        uint32_t q_cur = 0, n_cur = 0;
        {
            uint32_t upto = r.stage[0].group[0].count;
            while (k >= upto) { ++q_cur; upto += r.stage[0].group[q_cur].count; }
            next = upto < next ? upto : next;
        }
        for (uint32_t i = 0; i < P; ++i) {
            const sailor_mixed_stage& s = r.stage[i];
            const sailor_replica_group gr = s.group[q_cur];
            const uint32_t nb = base + (i < extra ? 1u : 0u);
            const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
            const size_t comp = (size_t)((e ? 2u : 0u) + (hd ? 1u : 0u)) * h->chain_len + nb;
            const double fb = v.cmp_fb[(((comp * T + gr.type) * h->n_tp + gr.tp_idx) * h->n_mbs + mi) * 2 + rc];
            double c = 0.0;
            if (i + 1 < P) {
                const sailor_mixed_stage& s2 = r.stage[i + 1];
                uint32_t q2 = 0, upto = s2.group[0].count;
                while (k >= upto) { ++q2; upto += s2.group[q2].count; }
                next = upto < next ? upto : next;
                const sailor_replica_group g2 = s2.group[q2];
                const uint32_t z = s.zone, z2 = s2.zone, g = gr.type;
                if (z != z2) {
                    c = link_time(v.zone_a[z * Z + z2], v.zone_i[z * Z + z2], v.zone_p, z * Z + z2, msg);
                } else if (g == g2.type && (uint64_t)gr.count * h->tp_values[gr.tp_idx] +
                                                   (uint64_t)g2.count * h->tp_values[g2.tp_idx] <= h->gpn[g]) {
                    const uint32_t d = z * T + g;
                    c = link_time(v.intra_a[d], v.intra_i[d], v.intra_p, d, msg);
                } else {
                    const uint32_t d = z * T + g, d2 = z * T + g2.type;
                    c = dmax(link_time(v.inter_a[d], v.inter_i[d], v.inter_p, d, msg),
                             link_time(v.inter_a[d2], v.inter_i[d2], v.inter_p, d2, msg));
                }
                n_cur = q2;
            }
            const double t = add_rn(fb, mul_rn(2.0, c));
            sum_t = add_rn(sum_t, t);
            max_t = dmax(max_t, t);
            q_cur = n_cur;
        }
        max_pp = dmax(max_pp, add_rn(sum_t, mul_rn((double)n_b, max_t)));
        k = next;
    }
    double c_comm = 0.0;
    const uint64_t xbytes = 2 * n_b * (uint64_t)D * v.p2p[mi];
    for (uint32_t i = 0; i + 1 < P; ++i) {
        const uint32_t z = r.stage[i].zone, z2 = r.stage[i + 1].zone;
        if (z != z2) c_comm = add_rn(c_comm, mul_rn((double)xbytes, v.egress[z * Z + z2]));
    }
    o.t_iter = add_rn(add_rn(max_pp, max_sync), max_u);
    o.cost = add_rn(mul_rn(rate, o.t_iter), c_comm);
    return o;
}

}  // namespace sailor
