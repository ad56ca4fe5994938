// Simulator for plans whose stages mix GPU types among their D replicas (Sailor Sec. 4.2, Sec. 4.3).
//
// Pipeline k runs on replica k of every stage, replicas being numbered group after group.  Two
// pipelines that use the same group in every stage are identical, so a plan has at most
// 1 + sum_i (groups_i - 1) different pipelines: the replica index is walked from one group boundary
// (of any stage) to the next, and one pipeline is evaluated per interval.  The arithmetic of one
// pipeline is the stage-by-stage evaluation of the plain simulator.
//
// One warp evaluates one plan, lane i owning stage i (and, in plans deeper than 32 stages, stages i + 32
// and i + 64): the per-stage terms of all stages are formed side by side, maxima are taken across the
// warp, and the sums whose order of additions is part of the result (stage times of a pipeline, price
// rate, transfer cost) are added up in stage order from the lanes' terms.  Plans differ widely in depth
// and in how many pipelines they have; a thread per plan kept four lanes of 32 busy on such batches.
#pragma once

#include "sailor_tables.cuh"

namespace sailor {

constexpr uint32_t MIX_FULL = 0xffffffffu;

// Largest of the warp's 64-bit values by two 32-bit warp maxima: the high words, then the low words of the lanes
// that hold the largest high word.
__device__ __forceinline__ uint64_t warp_max_u64(uint64_t x) {
    const uint32_t hi = (uint32_t)(x >> 32), lo = (uint32_t)x;
    const uint32_t mh = __reduce_max_sync(MIX_FULL, hi);
    const uint32_t ml = __reduce_max_sync(MIX_FULL, hi == mh ? lo : 0u);
    return (uint64_t)mh << 32 | ml;
}

// Largest of the warp's binary64 values (none is a NaN): the bit patterns, mapped so that unsigned order is numeric
// order (sign bit flipped for positive values, all bits for negative ones), go through warp_max_u64.
__device__ __forceinline__ double warp_max_f64(double x) {
    uint64_t b = (uint64_t)__double_as_longlong(x);
    b ^= (b >> 63) ? ~0ull : 0x8000000000000000ull;
    uint64_t m = warp_max_u64(b);
    m ^= (m >> 63) ? 0x8000000000000000ull : ~0ull;
    return __longlong_as_double((long long)m);
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
    if (P < 1 || P > 32 || D < 1 || mi >= h->n_mbs) return o;
    const bool mine = lane < P;

    // this lane's stage; group q as one word (type | tp_idx << 8 | count << 16), two words to a register pair, so
    // that the loops over a stage's groups need not be unrolled (the kernel waits on instruction fetch)
    uint32_t zone = 0, ng = 0;
    uint64_t g01 = 0, g23 = 0;
    auto group_word = [&](uint32_t q) { return (uint32_t)((q & 2u ? g23 : g01) >> (32u * (q & 1u))); };
    bool bad = false;
    if (mine) {
        const sailor_mixed_stage& s = r.stage[lane];
        zone = s.zone;
        ng = s.n_groups;
        bad = zone >= Z || ng < 1 || ng > SAILOR_MIX_GROUPS_MAX;
        if (!bad) {
            const uint32_t* g32 = reinterpret_cast<const uint32_t*>(&s.group[0]);      // a group is four bytes
            const uint32_t w0 = g32[0], w1 = ng > 1 ? g32[1] : 0u, w2 = ng > 2 ? g32[2] : 0u, w3 = ng > 3 ? g32[3] : 0u;
            g01 = (uint64_t)w0 | (uint64_t)w1 << 32;
            g23 = (uint64_t)w2 | (uint64_t)w3 << 32;
#pragma unroll 1
            for (uint32_t q = 0; q < ng; ++q) {
                const uint32_t gq = group_word(q);
                bad = bad || (gq & 0xff) >= T || ((gq >> 8) & 0xff) >= h->n_tp;
            }
        }
    }
    if (__any_sync(MIX_FULL, bad)) return o;

    uint32_t status = 0;
    const uint64_t dm = (uint64_t)D * h->mbs_values[mi];
    uint64_t n_b;
    if (((h->gbs | dm) >> 32) == 0) {                            // the usual case: a 32-bit division
        const uint32_t q32 = (uint32_t)h->gbs / (uint32_t)dm;
        n_b = q32;
        if (q32 * (uint32_t)dm != (uint32_t)h->gbs) status |= SAILOR_ST_INVALID;
    } else {
        n_b = h->gbs / dm;
        if (n_b * dm != h->gbs) status |= SAILOR_ST_INVALID;
    }
    const uint32_t base = h->n_blocks / P, extra = h->n_blocks - base * P;

    // validity, resources, memory per group, update time, synchronisation, price-rate terms: all stages at once
    for (uint32_t d = lane; d < R; d += 32) cnt[d] = 0;
    __syncwarp();
    const double steps = (double)(2 * (uint64_t)(D - 1));
    const double coef = steps / (double)D;
    double sync_l = 0.0, upd_l = 0.0;
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
#pragma unroll 1
        for (uint32_t q = 0; q < ng; ++q) {
            const uint32_t gq = group_word(q), ty = gq & 0xff, ti = (gq >> 8) & 0xff, cn = gq >> 16;
            const uint32_t tp = h->tp_values[ti];
            replicas += cn;
            if (cn == 0 || tp > h->gpn[ty] || h->heads % tp != 0) status |= SAILOR_ST_INVALID;
            atomicAdd(cnt + zone * T + ty, (unsigned long long)cn * tp);
            const size_t ct = comp * h->n_tp + ti;
            const uint64_t* mm = v.cmp_mem + ((ct * h->n_mbs + mi) * 2 + rc) * 2;
            const uint64_t m = mm[0] + inflight * mm[1] + h->reserved[ty];
            if (m > h->capacity[ty]) status |= SAILOR_ST_OOM;
            peak_l = m > peak_l ? m : peak_l;
            gradbytes = dmax(gradbytes, v.cmp_grad[ct]);          // the ring moves the largest shard (smallest tp)
        }
        if (replicas != D) status |= SAILOR_ST_INVALID;
#pragma unroll 1
        for (uint32_t q = 0; q < ng; ++q) {
            const uint32_t gq = group_word(q), ty = gq & 0xff, ti = (gq >> 8) & 0xff;
            const uint32_t d = zone * T + ty, tp = h->tp_values[ti];
            upd_l = dmax(upd_l, v.cmp_upd[(comp * T + ty) * h->n_tp + ti]);
            if (D > 1) {
                const bool intra = ng == 1 && (uint64_t)D * tp <= h->gpn[ty];
                sync_l = dmax(sync_l, allreduce_bytes_time(v, d, intra, gradbytes, D, steps, coef));
            }
        }
    }
    __syncwarp();                                                // the counters are complete
    if (mine) {
#pragma unroll 1
        for (uint32_t q = 0; q < ng; ++q) {
            const uint32_t d = zone * T + (group_word(q) & 0xff);
            if (cnt[d] > avail[d]) status |= SAILOR_ST_OVER_AVAIL;
        }
    }
    status = __reduce_or_sync(MIX_FULL, status);
    o.peak_mem = warp_max_u64(peak_l);
    o.status = status;
    if (status & SAILOR_ST_INVALID) return o;
    const double max_sync = warp_max_f64(sync_l), max_u = warp_max_f64(upd_l);
    double term[SAILOR_MIX_GROUPS_MAX];                          // this stage's price-rate terms
#pragma unroll
    for (uint32_t q = 0; q < SAILOR_MIX_GROUPS_MAX; ++q) {
        const uint32_t gq = group_word(q);                       // zero beyond the stage's groups: type 0, no replicas
        term[q] = mul_rn((double)((gq >> 16) * h->tp_values[(gq >> 8) & 0xff]), v.price_s[zone * T + (gq & 0xff)]);
    }
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
    const double msg = (double)v.p2p[mi];
    const uint32_t z2 = __shfl_down_sync(MIX_FULL, zone, 1);     // zone of the next stage
    const bool sends = mine && lane + 1 < P;
    double max_pp = 0.0;
    uint32_t k = 0;
    while (k < D) {
        // group of replica k in this lane's stage
        uint32_t cur = (uint32_t)g01, nxt = cur >> 16;
#pragma unroll
        for (uint32_t q = 1; q < SAILOR_MIX_GROUPS_MAX; ++q)
            if (q < ng && k >= nxt) { cur = group_word(q); nxt += cur >> 16; }
        const uint32_t g = cur & 0xff, tpi = (cur >> 8) & 0xff, cn = cur >> 16;
        const uint32_t next = __reduce_min_sync(MIX_FULL, mine ? nxt : D);
        const uint32_t cur2 = __shfl_down_sync(MIX_FULL, cur, 1);
        const uint32_t g2 = cur2 & 0xff, tpi2 = (cur2 >> 8) & 0xff, cn2 = cur2 >> 16;
        double t = 0.0;
        if (mine) {
            const double fb = v.cmp_fb[(((comp * T + g) * h->n_tp + tpi) * h->n_mbs + mi) * 2 + rc];
            double c = 0.0;
            if (sends) {
                // which link: its parameters are picked first, so that the link model is in the code once (twice for
                // the inter-node link between unlike types, whose slower end counts)
                const uint32_t z = zone, d = z * T + g;
                const bool cross = z != z2;
                const bool intra = !cross && g == g2 &&
                                   (uint64_t)cn * h->tp_values[tpi] + (uint64_t)cn2 * h->tp_values[tpi2] <= h->gpn[g];
                const uint32_t idx = cross ? z * Z + z2 : d;
                const double* la = cross ? v.zone_a : intra ? v.intra_a : v.inter_a;
                const double* li = cross ? v.zone_i : intra ? v.intra_i : v.inter_i;
                const double* lp = cross ? v.zone_p : intra ? v.intra_p : v.inter_p;
                c = link_time(la[idx], li[idx], lp, idx, msg);
                if (!cross && !intra && g2 != g) {
                    const uint32_t d2 = z * T + g2;
                    c = dmax(c, link_time(v.inter_a[d2], v.inter_i[d2], v.inter_p, d2, msg));
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

// The same evaluation for plans of up to 32 * TL stages: lane i owns stages i, i + 32, ... ("tiles").  A
// stage's groups are kept as packed words (type | tp_idx << 8 | count << 16); sums in stage order run
// through the tiles one after the other, and the stage after the last lane of a tile is the first lane of
// the next.
template <int TL>
__device__ __noinline__ SimOut simulate_mixed_tiles(const TabView& v, const uint16_t* __restrict__ avail,
                                                    const sailor_mixed_plan& r, unsigned long long* cnt, uint32_t lane) {
    static_assert(32 * TL <= SAILOR_MIX_P_MAX, "a record holds SAILOR_MIX_P_MAX stages");
    constexpr uint32_t G = SAILOR_MIX_GROUPS_MAX;
    const TabHdr* h = v.h;
    SimOut o;
    o.t_iter = o.cost = make_nan();
    o.peak_mem = 0;
    o.status = SAILOR_ST_BAD_RECORD;
    const uint32_t P = r.P, D = r.D, mi = r.mbs_idx, rc = r.rc ? 1u : 0u, T = h->T, Z = h->Z, R = h->R;
    if (P < 1 || P > 32 * TL || D < 1 || mi >= h->n_mbs) return o;

    uint32_t zone[TL], ng[TL], grp[TL][G];
    bool bad = false;
#pragma unroll
    for (int tl = 0; tl < TL; ++tl) {
        const uint32_t i = lane + 32 * tl;
        zone[tl] = ng[tl] = 0;
#pragma unroll
        for (uint32_t q = 0; q < G; ++q) grp[tl][q] = 0;
        if (i < P) {
            const sailor_mixed_stage& s = r.stage[i];
            zone[tl] = s.zone;
            ng[tl] = s.n_groups;
            bool b = zone[tl] >= Z || ng[tl] < 1 || ng[tl] > G;
#pragma unroll
            for (uint32_t q = 0; q < G; ++q)
                if (!b && q < ng[tl]) {
                    const uint32_t ty = s.group[q].type, ti = s.group[q].tp_idx;
                    if (ty >= T || ti >= h->n_tp) b = true;
                    grp[tl][q] = ty | ti << 8 | (uint32_t)s.group[q].count << 16;
                }
            bad = bad || b;
        }
    }
    if (__any_sync(MIX_FULL, bad)) return o;

    uint32_t status = 0;
    const uint64_t dm = (uint64_t)D * h->mbs_values[mi];
    if (h->gbs % dm != 0) status |= SAILOR_ST_INVALID;
    const uint64_t n_b = h->gbs / dm;
    const uint32_t base = h->n_blocks / P, extra = h->n_blocks % P;

    for (uint32_t d = lane; d < R; d += 32) cnt[d] = 0;
    __syncwarp();
    const double steps = (double)(2 * (uint64_t)(D - 1));
    const double coef = steps / (double)D;
    double sync_l = 0.0, upd_l = 0.0;
    uint64_t peak_l = 0;
    uint32_t comp[TL];
#pragma unroll
    for (int tl = 0; tl < TL; ++tl) {
        const uint32_t i = lane + 32 * tl;
        comp[tl] = 0;
        if (i < P) {
            const uint32_t nb = base + (i < extra ? 1u : 0u);
            const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
            const uint64_t inflight = (uint64_t)(P - i) < n_b ? (uint64_t)(P - i) : n_b;
            comp[tl] = ((e ? 2u : 0u) + (hd ? 1u : 0u)) * h->chain_len + nb;
            uint64_t replicas = 0;
            double gradbytes = 0.0;
#pragma unroll
            for (uint32_t q = 0; q < G; ++q)
                if (q < ng[tl]) {
                    const uint32_t ty = grp[tl][q] & 0xff, ti = (grp[tl][q] >> 8) & 0xff, cn = grp[tl][q] >> 16;
                    const uint32_t tp = h->tp_values[ti];
                    replicas += cn;
                    if (cn == 0 || tp > h->gpn[ty] || h->heads % tp != 0) status |= SAILOR_ST_INVALID;
                    atomicAdd(cnt + zone[tl] * T + ty, (unsigned long long)cn * tp);
                    const size_t ct = (size_t)comp[tl] * h->n_tp + ti;
                    const uint64_t* mm = v.cmp_mem + ((ct * h->n_mbs + mi) * 2 + rc) * 2;
                    const uint64_t m = mm[0] + inflight * mm[1] + h->reserved[ty];
                    if (m > h->capacity[ty]) status |= SAILOR_ST_OOM;
                    peak_l = m > peak_l ? m : peak_l;
                    gradbytes = dmax(gradbytes, v.cmp_grad[ct]);
                }
            if (replicas != D) status |= SAILOR_ST_INVALID;
#pragma unroll
            for (uint32_t q = 0; q < G; ++q)
                if (q < ng[tl]) {
                    const uint32_t ty = grp[tl][q] & 0xff, ti = (grp[tl][q] >> 8) & 0xff;
                    const uint32_t d = zone[tl] * T + ty, tp = h->tp_values[ti];
                    upd_l = dmax(upd_l, v.cmp_upd[((size_t)comp[tl] * T + ty) * h->n_tp + ti]);
                    if (D > 1) {
                        const bool intra = ng[tl] == 1 && (uint64_t)D * tp <= h->gpn[ty];
                        sync_l = dmax(sync_l, allreduce_bytes_time(v, d, intra, gradbytes, D, steps, coef));
                    }
                }
        }
    }
    __syncwarp();                                                // the counters are complete
#pragma unroll
    for (int tl = 0; tl < TL; ++tl)
#pragma unroll
        for (uint32_t q = 0; q < G; ++q)
            if (q < ng[tl]) {
                const uint32_t d = zone[tl] * T + (grp[tl][q] & 0xff);
                if (cnt[d] > avail[d]) status |= SAILOR_ST_OVER_AVAIL;
            }
    status = __reduce_or_sync(MIX_FULL, status);
    o.peak_mem = warp_max_u64(peak_l);
    o.status = status;
    if (status & SAILOR_ST_INVALID) return o;
    const double max_sync = warp_max_f64(sync_l), max_u = warp_max_f64(upd_l);
    double rate = 0.0;                                           // stage after stage, group after group
#pragma unroll
    for (int tl = 0; tl < TL; ++tl) {
        double term[G];
#pragma unroll
        for (uint32_t q = 0; q < G; ++q) {
            const uint32_t ty = grp[tl][q] & 0xff, ti = (grp[tl][q] >> 8) & 0xff, cn = grp[tl][q] >> 16;
            term[q] = q < ng[tl] ? mul_rn((double)(cn * h->tp_values[ti]), v.price_s[zone[tl] * T + ty]) : 0.0;
        }
        const uint32_t n_here = P > 32u * tl ? (P - 32u * tl < 32u ? P - 32u * tl : 32u) : 0u;
        for (uint32_t i = 0; i < n_here; ++i) {
            const uint32_t ng_i = __shfl_sync(MIX_FULL, ng[tl], i);
#pragma unroll
            for (uint32_t q = 0; q < G; ++q) {
                const double tq = __shfl_sync(MIX_FULL, term[q], i);
                if (q < ng_i) rate = add_rn(rate, tq);
            }
        }
    }

    // the pipelines
    uint32_t z2[TL];                                             // zone of the stage after this lane's
#pragma unroll
    for (int tl = 0; tl < TL; ++tl) {
        z2[tl] = __shfl_down_sync(MIX_FULL, zone[tl], 1);
        if (tl + 1 < TL) {
            const uint32_t first = __shfl_sync(MIX_FULL, zone[tl + 1 < TL ? tl + 1 : tl], 0);
            if (lane == 31) z2[tl] = first;
        }
    }
    const double msg = (double)v.p2p[mi];
    double max_pp = 0.0;
    uint32_t k = 0;
    while (k < D) {
        uint32_t cur[TL], nxt_l = D;                             // packed group of replica k, per tile
#pragma unroll
        for (int tl = 0; tl < TL; ++tl) {
            uint32_t run = grp[tl][0] >> 16, w = grp[tl][0];
#pragma unroll
            for (uint32_t q = 1; q < G; ++q)
                if (q < ng[tl] && k >= run) { w = grp[tl][q]; run += grp[tl][q] >> 16; }
            cur[tl] = w;
            if (lane + 32 * tl < P && run < nxt_l) nxt_l = run;
        }
        const uint32_t next = __reduce_min_sync(MIX_FULL, nxt_l);
        double t[TL];
#pragma unroll
        for (int tl = 0; tl < TL; ++tl) {
            uint32_t w2 = __shfl_down_sync(MIX_FULL, cur[tl], 1);
            if (tl + 1 < TL) {
                const uint32_t first = __shfl_sync(MIX_FULL, cur[tl + 1 < TL ? tl + 1 : tl], 0);
                if (lane == 31) w2 = first;
            }
            const uint32_t i = lane + 32 * tl;
            t[tl] = 0.0;
            if (i < P) {
                const uint32_t g = cur[tl] & 0xff, tpi = (cur[tl] >> 8) & 0xff, cn = cur[tl] >> 16;
                const uint32_t g2 = w2 & 0xff, tpi2 = (w2 >> 8) & 0xff, cn2 = w2 >> 16;
                const double fb = v.cmp_fb[((((size_t)comp[tl] * T + g) * h->n_tp + tpi) * h->n_mbs + mi) * 2 + rc];
                double c = 0.0;
                if (i + 1 < P) {
                    const uint32_t z = zone[tl], zn = z2[tl];
                    if (z != zn) {
                        c = link_time(v.zone_a[z * Z + zn], v.zone_i[z * Z + zn], v.zone_p, z * Z + zn, msg);
                    } else if (g == g2 && (uint64_t)cn * h->tp_values[tpi] + (uint64_t)cn2 * h->tp_values[tpi2] <= h->gpn[g]) {
                        const uint32_t d = z * T + g;
                        c = link_time(v.intra_a[d], v.intra_i[d], v.intra_p, d, msg);
                    } else {
                        const uint32_t d = z * T + g, d2 = z * T + g2;
                        c = dmax(link_time(v.inter_a[d], v.inter_i[d], v.inter_p, d, msg),
                                 link_time(v.inter_a[d2], v.inter_i[d2], v.inter_p, d2, msg));
                    }
                }
                t[tl] = add_rn(fb, mul_rn(2.0, c));
            }
        }
        double tm = t[0];
#pragma unroll
        for (int tl = 1; tl < TL; ++tl) tm = dmax(tm, t[tl]);
        const double max_t = warp_max_f64(tm);
        double sum_t = 0.0;                                      // in stage order
#pragma unroll
        for (int tl = 0; tl < TL; ++tl) {
            const uint32_t n_here = P > 32u * tl ? (P - 32u * tl < 32u ? P - 32u * tl : 32u) : 0u;
            for (uint32_t i = 0; i < n_here; ++i) sum_t = add_rn(sum_t, __shfl_sync(MIX_FULL, t[tl], i));
        }
        max_pp = dmax(max_pp, add_rn(sum_t, mul_rn((double)n_b, max_t)));
        k = next;
    }
    const uint64_t xbytes = 2 * n_b * (uint64_t)D * v.p2p[mi];
    double c_comm = 0.0;
#pragma unroll
    for (int tl = 0; tl < TL; ++tl) {
        const bool crosses = lane + 32 * tl + 1 < P && zone[tl] != z2[tl];
        const double cross_cost = crosses ? mul_rn((double)xbytes, v.egress[zone[tl] * Z + z2[tl]]) : 0.0;
        for (uint32_t m = __ballot_sync(MIX_FULL, crosses); m; m &= m - 1)    // boundaries in stage order
            c_comm = add_rn(c_comm, __shfl_sync(MIX_FULL, cross_cost, __ffs(m) - 1));
    }
    o.t_iter = add_rn(add_rn(max_pp, max_sync), max_u);
    o.cost = add_rn(mul_rn(rate, o.t_iter), c_comm);
    return o;
}

// Plans of up to 32 stages take the one-stage-per-lane evaluation, deeper ones the tiled one (the record's P
// is the same for every lane of the warp).
__device__ __forceinline__ SimOut simulate_mixed_plan(const TabView& v, const uint16_t* __restrict__ avail,
                                                      const sailor_mixed_plan& r, unsigned long long* cnt, uint32_t lane) {
    if (r.P <= 32) return simulate_mixed_warp(v, avail, r, cnt, lane);
    return simulate_mixed_tiles<SAILOR_MIX_P_MAX / 32>(v, avail, r, cnt, lane);
}

}  // namespace sailor
