/*
 * sailor_oracle.c — TEST INFRASTRUCTURE ONLY (see sailor_oracle.h).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -shared -fPIC
 * All times and costs are IEEE binary64, every sum runs left to right in stage order,
 * bytes and counts are 64-bit unsigned integers.
 */
#include "sailor_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

static uint64_t ceil_div_u64(uint64_t a, uint64_t b) { return (a + b - 1) / b; }
static uint64_t min_u64(uint64_t a, uint64_t b) { return a < b ? a : b; }
static double max_f64(double a, double b) { return a > b ? a : b; }

/* table lookups, index order as declared in orc_inputs */
static double tab4(const orc_inputs* in, const double* t, uint32_t kind, uint32_t g, uint32_t tp, uint32_t mbs) {
    return t[((kind * in->n_types + g) * in->n_tp + tp) * in->n_mbs + mbs];
}
static double tab_upd(const orc_inputs* in, uint32_t kind, uint32_t g, uint32_t tp) {
    return in->upd[(kind * in->n_types + g) * in->n_tp + tp];
}
static uint64_t tab_act(const orc_inputs* in, const uint64_t* t, uint32_t kind, uint32_t tp, uint32_t mbs) {
    return t[(kind * in->n_tp + tp) * in->n_mbs + mbs];
}

/* The layers of stage i of a P-stage pipeline, as a list of kinds.
 * Uniform split of the blocks, the remainder going one each to the first stages; the
 * embedding opens stage 0 and the head closes stage P-1 (Sec. 4.1: repeated layers are
 * profiled once, non-uniform ones separately). */
static uint32_t stage_layers(const orc_inputs* in, uint32_t P, uint32_t i, uint8_t* kinds) {
    uint32_t n = 0;
    uint32_t blocks = in->n_blocks / P + (i < in->n_blocks % P ? 1u : 0u);
    if (i == 0 && in->has_embed) kinds[n++] = 0;
    for (uint32_t j = 0; j < blocks; ++j) kinds[n++] = 1;
    if (i == P - 1 && in->has_head) kinds[n++] = 2;
    return n;
}

/* bandwidth of a link for a message of m bytes from its fitted polynomial (Sec. 4.1), Horner form */
static double poly_bw(const double* poly, double m) {
    return ((poly[3] * m + poly[2]) * m + poly[1]) * m + poly[0];
}
static const double* poly_at(const double* table, uint32_t idx) { return table ? table + 4 * idx : 0; }

/* time of one message of `bytes` over a link (Sec. 4.1: bandwidth depends on the message size).
 * With a fitted polynomial the time is alpha + m / bandwidth(m); without one it is the degree-1
 * time model alpha + m * inv_bw. */
static double link_time(double alpha, double inv_bw, const double* poly, uint64_t bytes) {
    double m = (double)bytes;
    if (poly) return alpha + m / poly_bw(poly, m);
    return alpha + m * inv_bw;
}

void orc_simulate(const orc_inputs* in, const orc_plan* pl, orc_out* out) {
    static uint8_t kinds[ORC_STAGES_MAX][1024 + 2];
    uint32_t nl[ORC_STAGES_MAX];
    const uint32_t P = pl->P, T = in->n_types, Z = in->n_zones;
    const uint32_t mbs_idx = pl->mbs_idx, D = pl->D, rc = pl->rc;
    const uint64_t mbs = in->mbs_values[mbs_idx];
    uint32_t status = 0;
    out->t_pp = out->t_sync = out->t_update = out->rate_per_s = out->c_comm = 0.0;

    /* validity: the global batch is never changed (Sec. 4.2), tensor parallelism stays in
     * one node (H1), attention heads split evenly */
    if (D == 0 || in->gbs % ((uint64_t)D * mbs) != 0) status |= ORC_INVALID;
    for (uint32_t i = 0; i < P; ++i) {
        uint32_t tp = in->tp_values[pl->tp_idx[i]];
        if (tp > in->gpus_per_node[pl->type[i]]) status |= ORC_INVALID;
        if (in->heads % tp != 0) status |= ORC_INVALID;
    }
    const uint64_t n_b = D ? in->gbs / ((uint64_t)D * mbs) : 0;
    out->n_b = n_b;

    /* resources: every stage takes D replicas of tp GPUs of its (zone, type) (H3: same D) */
    uint64_t used[64 * 64];
    memset(used, 0, sizeof(uint64_t) * Z * T);
    for (uint32_t i = 0; i < P; ++i)
        used[pl->zone[i] * T + pl->type[i]] += (uint64_t)D * in->tp_values[pl->tp_idx[i]];
    for (uint32_t d = 0; d < Z * T; ++d)
        if (used[d] > in->avail[d]) status |= ORC_OVER_AVAIL;

    /* memory per worker of each stage, Sec. 4.3: M_peak = M_model + M_activation */
    uint64_t params_stage[ORC_STAGES_MAX];
    uint64_t peak = 0;
    for (uint32_t i = 0; i < P; ++i) {
        nl[i] = stage_layers(in, P, i, kinds[i]);
        uint32_t g = pl->type[i], tpi = pl->tp_idx[i];
        uint64_t tp = in->tp_values[tpi];
        uint64_t params = 0, A = 0, W = 0;
        for (uint32_t l = 0; l < nl[i]; ++l) {
            uint32_t k = kinds[i][l];
            params += in->params[k];
            A += rc ? tab_act(in, in->act_ckpt, k, tpi, mbs_idx) : tab_act(in, in->act_saved, k, tpi, mbs_idx);
            uint64_t w = rc ? tab_act(in, in->act_saved, k, tpi, mbs_idx) : tab_act(in, in->act_work, k, tpi, mbs_idx);
            if (w > W) W = w;
        }
        params_stage[i] = params;
        uint64_t m_model = ceil_div_u64(params, tp) * in->mul_factor * in->dtype_size;
        uint64_t inflight = min_u64((uint64_t)(P - i), n_b);   /* 1F1B: stage i keeps P-i microbatches */
        uint64_t m = m_model + inflight * A + W + in->reserved[g];
        out->stage_mem[i] = m;
        if (m > in->capacity[g]) status |= ORC_OOM;
        if (m > peak) peak = m;
    }
    out->peak_mem = peak;
    out->status = status;
    if (status & ORC_INVALID) {
        out->t_iter = NAN;
        out->cost = NAN;
        return;
    }

    /* iteration time, Sec. 4.3: T_iter = max(T_pp) + T_sync + T_update, all pipelines alike */
    const uint64_t msg = in->p2p_bytes[mbs_idx];
    double sum_t = 0.0, max_t = 0.0, max_sync = 0.0, max_u = 0.0;
    for (uint32_t i = 0; i < P; ++i) {
        uint32_t g = pl->type[i], z = pl->zone[i], tpi = pl->tp_idx[i];
        uint32_t tp = in->tp_values[tpi];
        double f = 0.0, b = 0.0, u = 0.0;
        for (uint32_t l = 0; l < nl[i]; ++l) {
            uint32_t k = kinds[i][l];
            f = f + tab4(in, in->fwd, k, g, tpi, mbs_idx);
            b = b + tab4(in, in->bwd, k, g, tpi, mbs_idx);
            u = u + tab_upd(in, k, g, tpi);
        }
        if (rc) b = b + f;                 /* recomputation re-runs the forward pass */

        /* activation to the next stage and its gradient back over the same link */
        double c = 0.0;
        if (i + 1 < P) {
            uint32_t g2 = pl->type[i + 1], z2 = pl->zone[i + 1];
            uint32_t tp2 = in->tp_values[pl->tp_idx[i + 1]];
            if (z != z2) {
                c = link_time(in->zone_alpha[z * Z + z2], in->zone_inv_bw[z * Z + z2],
                              poly_at(in->zone_bw_poly, z * Z + z2), msg);
            } else if (g == g2 && (uint64_t)D * (tp + tp2) <= in->gpus_per_node[g]) {
                c = link_time(in->intra_alpha[z * T + g], in->intra_inv_bw[z * T + g],
                              poly_at(in->intra_bw_poly, z * T + g), msg);
            } else {
                double c1 = link_time(in->inter_alpha[z * T + g], in->inter_inv_bw[z * T + g],
                                      poly_at(in->inter_bw_poly, z * T + g), msg);
                double c2 = link_time(in->inter_alpha[z * T + g2], in->inter_inv_bw[z * T + g2],
                                      poly_at(in->inter_bw_poly, z * T + g2), msg);
                c = max_f64(c1, c2);
            }
        }
        double t = (f + b) + 2.0 * c;
        out->stage_c[i] = c;
        out->stage_t[i] = t;
        sum_t = sum_t + t;                 /* warm-up and cool-down: every stage once (Sec. 4.2.3) */
        max_t = max_f64(max_t, t);         /* the straggler sets the steady phase */
        max_u = max_f64(max_u, u);

        /* ring all-reduce of the stage's gradients among its D replicas, inside one zone (H5) */
        double sync = 0.0;
        if (D > 1) {
            uint64_t gradbytes = ceil_div_u64(params_stage[i], tp) * in->grad_dtype_size;
            double alpha, inv;
            const double* poly;
            if ((uint64_t)D * tp <= in->gpus_per_node[g]) {
                alpha = in->intra_alpha[z * T + g];
                inv = in->intra_inv_bw[z * T + g];
                poly = poly_at(in->intra_bw_poly, z * T + g);
            } else {
                alpha = in->inter_alpha[z * T + g];
                inv = in->inter_inv_bw[z * T + g];
                poly = poly_at(in->inter_bw_poly, z * T + g);
            }
            double steps = (double)(2 * (uint64_t)(D - 1));      /* ring: 2(D-1) messages of gradbytes/D */
            double coef = steps / (double)D;
            if (poly) {
                double chunk = (double)gradbytes / (double)D;
                sync = (coef * (double)gradbytes) / poly_bw(poly, chunk) + steps * alpha;
            } else {
                sync = (coef * (double)gradbytes) * inv + steps * alpha;
            }
        }
        out->stage_sync[i] = sync;
        max_sync = max_f64(max_sync, sync);
    }
    double t_pp = sum_t + (double)n_b * max_t;          /* T_total of Sec. 4.2.2 without sync */
    double t_iter = (t_pp + max_sync) + max_u;
    out->t_pp = t_pp;
    out->t_sync = max_sync;
    out->t_update = max_u;
    out->t_iter = t_iter;

    /* cost per iteration, Sec. 4.3: C_iter = C_comp + C_comm */
    double rate = 0.0;                                  /* dollars per second of all GPUs */
    for (uint32_t i = 0; i < P; ++i) {
        uint32_t n_gpus = D * in->tp_values[pl->tp_idx[i]];
        double per_s = in->price_per_hour[pl->zone[i] * T + pl->type[i]] / 3600.0;
        rate = rate + (double)n_gpus * per_s;
    }
    double c_comm = 0.0;
    for (uint32_t i = 0; i + 1 < P; ++i) {
        uint32_t z = pl->zone[i], z2 = pl->zone[i + 1];
        if (z != z2) {
            uint64_t bytes = 2 * n_b * (uint64_t)D * msg;    /* forward and backward, all microbatches, all replicas */
            c_comm = c_comm + (double)bytes * in->egress[z * Z + z2];
        }
    }
    out->rate_per_s = rate;
    out->c_comm = c_comm;
    out->cost = rate * t_iter + c_comm;
}

static uint64_t ipow_u64(uint64_t b, uint32_t e) {
    uint64_t r = 1;
    while (e--) r *= b;
    return r;
}
static uint32_t nseg_of(const orc_space* sp, uint32_t P) { return P < sp->seg_max ? P : sp->seg_max; }

uint64_t orc_space_size(const orc_inputs* in, const orc_space* sp) {
    uint64_t radix = (uint64_t)in->n_types * in->n_zones;
    uint64_t base = (uint64_t)sp->n_mbs * sp->n_tp * sp->n_rc * sp->n_d;
    uint64_t n = 0;
    for (uint32_t j = 0; j < sp->n_p; ++j) n += base * ipow_u64(radix, nseg_of(sp, sp->p_values[j]));
    return n;
}

/* Flat index -> plan.  The sub-spaces of the P values follow one another; inside one, the
 * digits from the lowest are: segment nseg-1 ... segment 0 (radix T*Z, digit = zone*T+type),
 * D, recomputation, tp, mbs.  Stage i takes segment floor(i*nseg/P). */
int orc_decode(const orc_inputs* in, const orc_space* sp, uint64_t flat, orc_plan* pl) {
    uint64_t radix = (uint64_t)in->n_types * in->n_zones;
    uint64_t base = (uint64_t)sp->n_mbs * sp->n_tp * sp->n_rc * sp->n_d;
    for (uint32_t j = 0; j < sp->n_p; ++j) {
        uint32_t P = sp->p_values[j];
        uint32_t nseg = nseg_of(sp, P);
        uint64_t sub = base * ipow_u64(radix, nseg);
        if (flat >= sub) { flat -= sub; continue; }
        uint32_t seg[ORC_SEG_MAX];
        for (uint32_t s = nseg; s-- > 0;) { seg[s] = (uint32_t)(flat % radix); flat /= radix; }
        uint32_t di = (uint32_t)(flat % sp->n_d);   flat /= sp->n_d;
        uint32_t ri = (uint32_t)(flat % sp->n_rc);  flat /= sp->n_rc;
        uint32_t ti = (uint32_t)(flat % sp->n_tp);  flat /= sp->n_tp;
        uint32_t mi = (uint32_t)flat;
        pl->P = P;
        pl->mbs_idx = sp->mbs_idx[mi];
        pl->rc = sp->rc_values[ri];
        pl->D = sp->d_values[di];
        for (uint32_t i = 0; i < P; ++i) {
            uint32_t s = (uint32_t)(((uint64_t)i * nseg) / P);
            pl->type[i] = seg[s] % in->n_types;
            pl->zone[i] = seg[s] / in->n_types;
            pl->tp_idx[i] = sp->tp_idx[ti];
        }
        return 0;
    }
    return -1;
}

static int hit_before(const orc_hit* a, double score, uint64_t flat) {
    return a->score < score || (a->score == score && a->flat < flat);
}

/* sorted insertion: (score, flat) ascending, keep k (Sec. 4.2: sort by objective); returns the new length */
static uint32_t offer_hit(orc_hit* hits, uint32_t n_hits, uint32_t k, uint64_t flat, double score, const orc_out* o) {
    if (k == 0) return n_hits;
    if (n_hits == k && hit_before(&hits[k - 1], score, flat)) return n_hits;
    uint32_t pos = n_hits < k ? n_hits : k - 1;
    while (pos > 0 && !hit_before(&hits[pos - 1], score, flat)) {
        hits[pos] = hits[pos - 1];
        pos--;
    }
    hits[pos].flat = flat;
    hits[pos].score = score;
    hits[pos].t_iter = o->t_iter;
    hits[pos].cost = o->cost;
    hits[pos].peak_mem = o->peak_mem;
    return n_hits < k ? n_hits + 1 : n_hits;
}

uint32_t orc_search(const orc_inputs* in, const orc_space* sp, const orc_objective* obj,
                    uint64_t lo, uint64_t hi, uint64_t stride, uint32_t k, orc_hit* hits,
                    orc_counts* counts) {
    orc_plan pl;
    orc_out o;
    uint32_t n_hits = 0;
    orc_counts c;
    memset(&c, 0, sizeof(c));
    if (stride == 0) stride = 1;
    for (uint64_t flat = lo; flat < hi; flat += stride) {
        if (orc_decode(in, sp, flat, &pl) != 0) break;
        orc_simulate(in, &pl, &o);
        c.n_total++;
        if (o.status & ORC_INVALID) { c.n_invalid++; continue; }
        if (o.status & ORC_OOM) { c.n_oom++; continue; }
        if (o.status & ORC_OVER_AVAIL) { c.n_over_avail++; continue; }
        /* the planner keeps a configuration only when it is within the constraint (Sec. 4.2) */
        int over = 0;
        if (obj->budget > 0.0 && o.cost > obj->budget) over = 1;
        if (obj->min_rate > 0.0 && 1.0 / o.t_iter < obj->min_rate) over = 1;
        if (over) { c.n_over_constraint++; continue; }
        c.n_feasible++;
        if (c.n_feasible == 1 || o.cost < c.min_cost) c.min_cost = o.cost;
        double score = obj->kind == ORC_OBJ_TIME ? o.t_iter
                     : obj->kind == ORC_OBJ_COST ? o.cost
                                                 : o.t_iter * o.cost;
        n_hits = offer_hit(hits, n_hits, k, flat, score, &o);
    }
    if (counts) *counts = c;
    return n_hits;
}

void orc_simulate_flat(const orc_inputs* in, const orc_space* sp, const uint64_t* flat, uint64_t n,
                       uint32_t* status, double* t_iter, double* cost, uint64_t* peak_mem) {
    orc_plan pl;
    orc_out o;
    for (uint64_t j = 0; j < n; ++j) {
        if (orc_decode(in, sp, flat[j], &pl) != 0) { status[j] = 0xFFFFFFFFu; continue; }
        orc_simulate(in, &pl, &o);
        status[j] = o.status;
        t_iter[j] = o.t_iter;
        cost[j] = o.cost;
        peak_mem[j] = o.peak_mem;
    }
}

void orc_simulate_batch(const orc_inputs* in, const orc_plan* plans, uint64_t n,
                        uint32_t* status, double* t_iter, double* cost, uint64_t* peak_mem) {
    orc_out o;
    for (uint64_t j = 0; j < n; ++j) {
        orc_simulate(in, &plans[j], &o);
        status[j] = o.status;
        t_iter[j] = o.t_iter;
        cost[j] = o.cost;
        peak_mem[j] = o.peak_mem;
    }
}

/* ---- the planner's pruning heuristics as search modes (Sec. 4.2.1) ------------------------------- */

static double score_of(const orc_objective* obj, const orc_out* o) {
    return obj->kind == ORC_OBJ_TIME ? o->t_iter : obj->kind == ORC_OBJ_COST ? o->cost : o->t_iter * o->cost;
}

/* H2, taken one step further than the paper's wording (which only drops tensor-parallel degrees that do
 * not fit): is there a smaller degree in the space's list at which this very plan is valid and every
 * stage fits in memory?  Then the plan is not the minimum-degree one and the mode drops it. */
static int fits_with_smaller_tp(const orc_inputs* in, const orc_space* sp, const orc_plan* pl, uint32_t ti) {
    const uint32_t tp = in->tp_values[sp->tp_idx[ti]];
    for (uint32_t tj = 0; tj < sp->n_tp; ++tj) {
        if (in->tp_values[sp->tp_idx[tj]] >= tp) continue;
        orc_plan q = *pl;
        for (uint32_t i = 0; i < q.P; ++i) q.tp_idx[i] = sp->tp_idx[tj];
        orc_out o;
        orc_simulate(in, &q, &o);
        if (!(o.status & (ORC_INVALID | ORC_OOM))) return 1;
    }
    return 0;
}

int32_t orc_search_pruned(const orc_inputs* in, const orc_space* sp, const orc_objective* obj, uint32_t modes,
                          uint32_t k, orc_hit* hits, orc_pruned_counts* counts) {
    orc_pruned_counts c;
    memset(&c, 0, sizeof(c));
    if ((modes & ORC_PRUNE_D_ORDER) && obj->kind != ORC_OBJ_TIME && obj->kind != ORC_OBJ_COST) return -1;
    const uint64_t radix = (uint64_t)in->n_types * in->n_zones;
    const uint64_t base = (uint64_t)sp->n_mbs * sp->n_tp * sp->n_rc * sp->n_d;

    /* the order in which a group's data-parallel degrees are tried: largest first when throughput is
     * maximised (H3), smallest first when cost is minimised (H4); without the mode, as listed */
    uint32_t order[256];
    if (sp->n_d > 256) return -1;
    for (uint32_t j = 0; j < sp->n_d; ++j) order[j] = j;
    if (modes & ORC_PRUNE_D_ORDER) {
        const int descending = obj->kind == ORC_OBJ_TIME;
        for (uint32_t a = 1; a < sp->n_d; ++a) {             /* insertion sort, stable */
            uint32_t x = order[a], b = a;
            while (b > 0 && (descending ? sp->d_values[order[b - 1]] < sp->d_values[x]
                                        : sp->d_values[order[b - 1]] > sp->d_values[x])) {
                order[b] = order[b - 1];
                b--;
            }
            order[b] = x;
        }
    }

    uint32_t n_hits = 0;
    uint64_t p_base = 0;                                     /* flat index of the sub-space of this P */
    orc_plan pl;
    orc_out o;
    for (uint32_t jp = 0; jp < sp->n_p; ++jp) {
        const uint32_t P = sp->p_values[jp];
        const uint64_t per_cfg = ipow_u64(radix, nseg_of(sp, P));
        for (uint32_t mi = 0; mi < sp->n_mbs; ++mi)
        for (uint32_t ti = 0; ti < sp->n_tp; ++ti)
        for (uint32_t ri = 0; ri < sp->n_rc; ++ri) {
            /* one group: everything fixed but the data-parallel degree */
            int have_prev = 0, stopped = 0;
            double prev_best = 0.0;
            for (uint32_t step = 0; step < sp->n_d; ++step) {
                const uint32_t di = order[step];
                c.n_configs++;
                if (stopped) { c.n_skipped += per_cfg; continue; }
                c.n_configs_evaluated++;
                const uint64_t first = p_base + ((((uint64_t)mi * sp->n_tp + ti) * sp->n_rc + ri) * sp->n_d + di) * per_cfg;
                int have_best = 0;
                double best = 0.0;
                for (uint64_t flat = first; flat < first + per_cfg; ++flat) {
                    if (orc_decode(in, sp, flat, &pl) != 0) return -1;
                    orc_simulate(in, &pl, &o);
                    c.looked_at.n_total++;
                    if (o.status & ORC_INVALID) { c.looked_at.n_invalid++; continue; }
                    if (o.status & ORC_OOM) { c.looked_at.n_oom++; continue; }
                    if ((modes & ORC_PRUNE_MIN_TP) && fits_with_smaller_tp(in, sp, &pl, ti)) { c.n_pruned_tp++; continue; }
                    if (o.status & ORC_OVER_AVAIL) { c.looked_at.n_over_avail++; continue; }
                    int over = 0;
                    if (obj->budget > 0.0 && o.cost > obj->budget) over = 1;
                    if (obj->min_rate > 0.0 && 1.0 / o.t_iter < obj->min_rate) over = 1;
                    if (over) { c.looked_at.n_over_constraint++; continue; }
                    c.looked_at.n_feasible++;
                    if (c.looked_at.n_feasible == 1 || o.cost < c.looked_at.min_cost) c.looked_at.min_cost = o.cost;
                    const double score = score_of(obj, &o);
                    if (!have_best || score < best) { best = score; have_best = 1; }
                    n_hits = offer_hit(hits, n_hits, k, flat, score, &o);
                }
                if (!(modes & ORC_PRUNE_D_ORDER)) continue;
                /* H3 / H4: degrees without a feasible plan are passed over until the first feasible one is
                 * found; from then on the next degree is tried only while the group's best objective
                 * improved strictly */
                if (!have_best) { if (have_prev) stopped = 1; continue; }
                if (have_prev && !(best < prev_best)) { stopped = 1; continue; }
                prev_best = best;
                have_prev = 1;
            }
        }
        p_base += base * per_cfg;
    }
    if (counts) *counts = c;
    return (int32_t)n_hits;
}

/* ---- per-stage resource assignment by dynamic programming (Sec. 4.2.2, Eq. 1 and the listing) ------
 *
 * Everything of a plan is fixed but the GPU type of each stage: P, mbs, tp, recomputation, D, and the
 * order in which the zones are filled.  Stage i takes D replicas of tp GPUs of one type g_i and is placed
 * by first fit: the first zone, at or after the zone of stage i-1 in the given order, that still has
 * D*tp GPUs of that type free.  The recursion gives stage i its resources, solves stages i+1.. on what
 * is left, and combines the two by T_total (straggler * N_b + slowest synchronisation + sum of the stage
 * times, and the slowest update as in Sec. 4.3); it keeps the best and remembers it per state.  As in the
 * paper the rest of the pipeline is solved on its own, so the result is the best plan among those whose
 * every suffix is the best one for its state: an approximation of the optimum, not the optimum.
 */

/* the quantities of one stage that the simulator adds up, computed the same way (layer by layer) */
static void dp_stage(const orc_inputs* in, uint32_t P, uint32_t i, uint32_t g, uint32_t tpi, uint32_t mbs_idx,
                     uint32_t rc, uint64_t n_b, double* fb, double* upd, uint64_t* params, int* fits) {
    uint8_t kinds[1024 + 2];
    const uint32_t nl = stage_layers(in, P, i, kinds);
    const uint64_t tp = in->tp_values[tpi];
    double f = 0.0, b = 0.0, u = 0.0;
    uint64_t par = 0, A = 0, W = 0;
    for (uint32_t l = 0; l < nl; ++l) {
        const uint32_t k = kinds[l];
        f = f + tab4(in, in->fwd, k, g, tpi, mbs_idx);
        b = b + tab4(in, in->bwd, k, g, tpi, mbs_idx);
        u = u + tab_upd(in, k, g, tpi);
        par += in->params[k];
        A += rc ? tab_act(in, in->act_ckpt, k, tpi, mbs_idx) : tab_act(in, in->act_saved, k, tpi, mbs_idx);
        const uint64_t w = rc ? tab_act(in, in->act_saved, k, tpi, mbs_idx) : tab_act(in, in->act_work, k, tpi, mbs_idx);
        if (w > W) W = w;
    }
    if (rc) b = b + f;
    *fb = f + b;
    *upd = u;
    *params = par;
    const uint64_t m = ceil_div_u64(par, tp) * in->mul_factor * in->dtype_size + min_u64((uint64_t)(P - i), n_b) * A + W +
                       in->reserved[g];
    *fits = m <= in->capacity[g] && tp <= in->gpus_per_node[g];
}

/* one message from a stage on (g, z) to the next stage on (g2, z2), both with degree tp */
static double dp_p2p(const orc_inputs* in, uint32_t g, uint32_t z, uint32_t g2, uint32_t z2, uint32_t tp, uint32_t D,
                     uint64_t msg) {
    const uint32_t T = in->n_types, Z = in->n_zones;
    if (z != z2)
        return link_time(in->zone_alpha[z * Z + z2], in->zone_inv_bw[z * Z + z2], poly_at(in->zone_bw_poly, z * Z + z2), msg);
    if (g == g2 && (uint64_t)D * (tp + tp) <= in->gpus_per_node[g])
        return link_time(in->intra_alpha[z * T + g], in->intra_inv_bw[z * T + g], poly_at(in->intra_bw_poly, z * T + g), msg);
    const double c1 = link_time(in->inter_alpha[z * T + g], in->inter_inv_bw[z * T + g], poly_at(in->inter_bw_poly, z * T + g), msg);
    const double c2 = link_time(in->inter_alpha[z * T + g2], in->inter_inv_bw[z * T + g2], poly_at(in->inter_bw_poly, z * T + g2), msg);
    return max_f64(c1, c2);
}

/* ring all-reduce of a stage's gradients among its D replicas on (g, z) */
static double dp_sync(const orc_inputs* in, uint32_t g, uint32_t z, uint32_t tp, uint32_t D, uint64_t params) {
    if (D <= 1) return 0.0;
    const uint32_t T = in->n_types, d = z * T + g;
    const uint64_t gradbytes = ceil_div_u64(params, tp) * in->grad_dtype_size;
    const int intra = (uint64_t)D * tp <= in->gpus_per_node[g];
    const double alpha = intra ? in->intra_alpha[d] : in->inter_alpha[d];
    const double inv = intra ? in->intra_inv_bw[d] : in->inter_inv_bw[d];
    const double* poly = intra ? poly_at(in->intra_bw_poly, d) : poly_at(in->inter_bw_poly, d);
    const double steps = (double)(2 * (uint64_t)(D - 1));
    const double coef = steps / (double)D;
    if (poly) return (coef * (double)gradbytes) / poly_bw(poly, (double)gradbytes / (double)D) + steps * alpha;
    return (coef * (double)gradbytes) * inv + steps * alpha;
}

typedef struct dp_val {
    int state;                 /* 0 not computed, 1 no plan, 2 plan */
    int next_g;                /* type of the next stage in the kept plan */
    double sum, mx, sy, up;    /* sum of stage times, straggler, slowest synchronisation, slowest update */
} dp_val;

typedef struct dp_key { uint64_t used; uint32_t igz; } dp_key;       /* used: one byte per type; igz: stage, type, zone position */

typedef struct dp_ctx {
    const orc_inputs* in;
    const orc_dp_problem* pb;
    uint32_t T, need, tp;
    uint64_t n_b, msg;
    int use_memo;
    /* per (stage, type) */
    double fb[ORC_STAGES_MAX][ORC_DP_T_MAX], upd[ORC_STAGES_MAX][ORC_DP_T_MAX];
    uint64_t params[ORC_STAGES_MAX];
    int fits[ORC_STAGES_MAX][ORC_DP_T_MAX];
    /* memo: open addressing */
    dp_key* keys; dp_val* vals; uint8_t* full; uint64_t cap, count;
    uint64_t n_states;
} dp_ctx;

static double dp_value(const dp_ctx* c, const dp_val* v) {
    return ((v->sum + (double)c->n_b * v->mx) + v->sy) + v->up;
}

static uint64_t dp_hash(dp_key k) {
    uint64_t x = k.used * 0x9E3779B97F4A7C15ull ^ ((uint64_t)k.igz * 0xBF58476D1CE4E5B9ull);
    x ^= x >> 29;
    return x * 0x94D049BB133111EBull;
}

static dp_val* memo_slot(dp_ctx* c, dp_key k) {
    if ((c->count + 1) * 2 > c->cap) {                       /* grow and reinsert */
        const uint64_t ncap = c->cap ? c->cap * 2 : 1024;
        dp_key* nk = (dp_key*)calloc(ncap, sizeof(dp_key));
        dp_val* nv = (dp_val*)calloc(ncap, sizeof(dp_val));
        uint8_t* nf = (uint8_t*)calloc(ncap, 1);
        for (uint64_t j = 0; j < c->cap; ++j) {
            if (!c->full[j]) continue;
            uint64_t h = dp_hash(c->keys[j]) & (ncap - 1);
            while (nf[h]) h = (h + 1) & (ncap - 1);
            nk[h] = c->keys[j]; nv[h] = c->vals[j]; nf[h] = 1;
        }
        free(c->keys); free(c->vals); free(c->full);
        c->keys = nk; c->vals = nv; c->full = nf; c->cap = ncap;
    }
    uint64_t h = dp_hash(k) & (c->cap - 1);
    while (c->full[h]) {
        if (c->keys[h].used == k.used && c->keys[h].igz == k.igz) return &c->vals[h];
        h = (h + 1) & (c->cap - 1);
    }
    c->full[h] = 1;
    c->keys[h] = k;
    memset(&c->vals[h], 0, sizeof(dp_val));
    c->count++;
    return &c->vals[h];
}

/* first zone position at or after `zp` with D*tp GPUs of type g free; `used` counts the stages already
 * placed in zone position zp, per type (later zones are untouched, earlier ones are not revisited) */
static int first_fit(const dp_ctx* c, uint32_t zp, const uint8_t* used, uint32_t g) {
    for (uint32_t p = zp; p < c->pb->n_zones_used; ++p) {
        const uint64_t have = c->in->avail[c->pb->zone_list[p] * c->T + g];
        const uint64_t taken = (p == zp) ? (uint64_t)used[g] * c->need : 0;
        if (have >= taken + c->need) return (int)p;
    }
    return -1;
}

/* best plan for stages i.. given that stage i runs on type g in zone position zp and `used` (which
 * includes stage i) describes that zone */
static dp_val solve_suffix(dp_ctx* c, uint32_t i, uint32_t g, uint32_t zp, const uint8_t* used) {
    const uint32_t P = c->pb->P, z = c->pb->zone_list[zp];
    dp_val none; memset(&none, 0, sizeof(none)); none.state = 1; none.next_g = -1;
    if (!c->fits[i][g]) return none;
    dp_key key; key.used = 0; key.igz = (i << 8) | (g << 4) | zp;
    for (uint32_t t = 0; t < c->T; ++t) key.used |= (uint64_t)used[t] << (8 * t);
    if (c->use_memo) {
        dp_val* slot = memo_slot(c, key);
        if (slot->state) return *slot;
    }
    c->n_states++;
    dp_val best = none;
    const double sync = dp_sync(c->in, g, z, c->tp, c->pb->D, c->params[i]);
    if (i == P - 1) {
        best.state = 2;
        best.sum = c->fb[i][g];                  /* the last stage sends nothing */
        best.mx = c->fb[i][g];
        best.sy = sync;
        best.up = c->upd[i][g];
    } else {
        for (uint32_t g2 = 0; g2 < c->T; ++g2) {
            if (!c->fits[i + 1][g2]) continue;
            const int zp2 = first_fit(c, zp, used, g2);
            if (zp2 < 0) continue;
            uint8_t used2[ORC_DP_T_MAX];
            for (uint32_t t = 0; t < c->T; ++t) used2[t] = ((uint32_t)zp2 == zp) ? used[t] : 0;
            used2[g2]++;
            const dp_val nxt = solve_suffix(c, i + 1, g2, (uint32_t)zp2, used2);
            if (nxt.state != 2) continue;
            const double cmsg = dp_p2p(c->in, g, z, g2, c->pb->zone_list[zp2], c->tp, c->pb->D, c->msg);
            const double t = c->fb[i][g] + 2.0 * cmsg;
            dp_val cand;
            cand.state = 2;
            cand.next_g = (int)g2;
            cand.sum = t + nxt.sum;
            cand.mx = max_f64(t, nxt.mx);
            cand.sy = max_f64(sync, nxt.sy);
            cand.up = max_f64(c->upd[i][g], nxt.up);
            if (best.state != 2 || dp_value(c, &cand) < dp_value(c, &best)) best = cand;
        }
    }
    if (c->use_memo) *memo_slot(c, key) = best;
    return best;
}

int orc_solve_dp(const orc_inputs* in, const orc_dp_problem* pb, int use_memo, orc_dp_result* out) {
    memset(out, 0, sizeof(*out));
    const uint32_t P = pb->P, T = in->n_types;
    if (P < 1 || P > ORC_STAGES_MAX || T > ORC_DP_T_MAX || pb->n_zones_used < 1 || pb->n_zones_used > 16 || pb->D < 1) return -1;
    const uint64_t mbs = in->mbs_values[pb->mbs_idx];
    const uint32_t tp = in->tp_values[pb->tp_idx];
    if (in->gbs % ((uint64_t)pb->D * mbs) != 0 || in->heads % tp != 0) return 0;      /* no valid plan in this problem */
    dp_ctx* c = (dp_ctx*)calloc(1, sizeof(dp_ctx));
    c->in = in; c->pb = pb; c->T = T; c->tp = tp; c->need = pb->D * tp;
    c->n_b = in->gbs / ((uint64_t)pb->D * mbs);
    c->msg = in->p2p_bytes[pb->mbs_idx];
    c->use_memo = use_memo;
    for (uint32_t i = 0; i < P; ++i)
        for (uint32_t g = 0; g < T; ++g) {
            uint64_t par;
            dp_stage(in, P, i, g, pb->tp_idx, pb->mbs_idx, pb->rc, c->n_b, &c->fb[i][g], &c->upd[i][g], &par, &c->fits[i][g]);
            c->params[i] = par;
        }
    /* stage 0: every type, placed by first fit from the first zone of the order */
    dp_val best; memset(&best, 0, sizeof(best)); best.state = 1;
    int best_g = -1, best_zp = -1;
    const uint8_t nothing[ORC_DP_T_MAX] = {0};
    for (uint32_t g = 0; g < T; ++g) {
        const int zp = first_fit(c, 0, nothing, g);
        if (zp < 0) continue;
        uint8_t used[ORC_DP_T_MAX] = {0};
        used[g] = 1;
        const dp_val v = solve_suffix(c, 0, g, (uint32_t)zp, used);
        if (v.state != 2) continue;
        if (best.state != 2 || dp_value(c, &v) < dp_value(c, &best)) { best = v; best_g = (int)g; best_zp = zp; }
    }
    out->n_states = c->n_states;
    if (best.state == 2) {
        out->found = 1;
        out->value = dp_value(c, &best);
        /* walk the kept choices to write the plan out */
        orc_plan* pl = &out->plan;
        pl->P = P; pl->mbs_idx = pb->mbs_idx; pl->rc = pb->rc; pl->D = pb->D;
        uint8_t used[ORC_DP_T_MAX] = {0};
        uint32_t g = (uint32_t)best_g, zp = (uint32_t)best_zp;
        used[g] = 1;
        dp_val v = best;
        for (uint32_t i = 0; i < P; ++i) {
            pl->type[i] = g; pl->zone[i] = pb->zone_list[zp]; pl->tp_idx[i] = pb->tp_idx;
            if (i + 1 == P) break;
            const uint32_t g2 = (uint32_t)v.next_g;
            const int zp2 = first_fit(c, zp, used, g2);
            if ((uint32_t)zp2 != zp) memset(used, 0, sizeof(used));
            used[g2]++;
            g = g2; zp = (uint32_t)zp2;
            v = solve_suffix(c, i + 1, g, zp, used);
        }
    }
    free(c->keys); free(c->vals); free(c->full); free(c);
    return 0;
}

/* ---- the recursion under a cost limit (Sec. 4.2.3) ---------------------------------------------------- */

typedef struct dpb_val {
    int found;
    double sum, mx, sy, up;              /* as dp_val */
    double cost;                         /* what stages i.. were charged */
    uint8_t type[ORC_STAGES_MAX];        /* types of stages i.. of the kept plan, at their own positions */
} dpb_val;

static double dpb_value(const dp_ctx* c, const dpb_val* v) {
    return ((v->sum + (double)c->n_b * v->mx) + v->sy) + v->up;
}

/* best plan within `limit` for stages i.. given that stage i runs on type g in zone position zp and `used`
 * (which includes stage i) describes that zone */
static dpb_val solve_suffix_budget(dp_ctx* c, uint32_t i, uint32_t g, uint32_t zp, const uint8_t* used, double limit) {
    const orc_inputs* in = c->in;
    const uint32_t P = c->pb->P, z = c->pb->zone_list[zp], D = c->pb->D;
    dpb_val best; memset(&best, 0, sizeof(best));
    if (!c->fits[i][g]) return best;
    c->n_states++;
    const double sync = dp_sync(in, g, z, c->tp, D, c->params[i]);
    const double rate = (double)(D * c->tp) * (in->price_per_hour[z * c->T + g] / 3600.0);
    if (i == P - 1) {
        const double t = c->fb[i][g];                        /* the last stage sends nothing and is its own straggler */
        const double charge = rate * ((double)c->n_b * t);
        if (charge <= limit) {
            best.found = 1;
            best.sum = t; best.mx = t; best.sy = sync; best.up = c->upd[i][g];
            best.cost = charge;
            best.type[i] = (uint8_t)g;
        }
        return best;
    }
    for (uint32_t g2 = 0; g2 < c->T; ++g2) {
        if (!c->fits[i + 1][g2]) continue;
        const int zp2 = first_fit(c, zp, used, g2);
        if (zp2 < 0) continue;
        uint8_t used2[ORC_DP_T_MAX];
        for (uint32_t t = 0; t < c->T; ++t) used2[t] = ((uint32_t)zp2 == zp) ? used[t] : 0;
        used2[g2]++;
        const uint32_t z2 = c->pb->zone_list[zp2];
        const double cmsg = dp_p2p(in, g, z, g2, z2, c->tp, D, c->msg);
        const double t = c->fb[i][g] + 2.0 * cmsg;
        const double comm = (z2 != z) ? (double)(2 * c->n_b * (uint64_t)D * c->msg) * in->egress[z * in->n_zones + z2] : 0.0;
        double assumed = t;                                  /* first: this stage is the straggler */
        for (;;) {
            const double charge = rate * ((double)c->n_b * assumed) + comm;
            const double rest = limit - charge;
            if (!(rest > 0.0)) break;
            const dpb_val nxt = solve_suffix_budget(c, i + 1, g2, (uint32_t)zp2, used2, rest);
            if (!nxt.found) break;
            if (nxt.mx <= assumed) {                         /* the assumption holds */
                const double all = charge + nxt.cost;
                if (all <= limit) {
                    dpb_val cand = nxt;                      /* keeps the types of the later stages */
                    cand.found = 1;
                    cand.sum = t + nxt.sum;
                    cand.mx = max_f64(t, nxt.mx);
                    cand.sy = max_f64(sync, nxt.sy);
                    cand.up = max_f64(c->upd[i][g], nxt.up);
                    cand.cost = all;
                    cand.type[i] = (uint8_t)g;
                    if (!best.found || dpb_value(c, &cand) < dpb_value(c, &best)) best = cand;
                }
                break;
            }
            assumed = nxt.mx;                                /* charge again with the straggler that was found */
        }
    }
    return best;
}

int orc_solve_dp_budget(const orc_inputs* in, const orc_dp_problem* pb, double limit, orc_dp_budget_result* out) {
    memset(out, 0, sizeof(*out));
    const uint32_t P = pb->P, T = in->n_types;
    if (P < 1 || P > ORC_STAGES_MAX || T > ORC_DP_T_MAX || pb->n_zones_used < 1 || pb->n_zones_used > 16 || pb->D < 1) return -1;
    const uint64_t mbs = in->mbs_values[pb->mbs_idx];
    const uint32_t tp = in->tp_values[pb->tp_idx];
    if (in->gbs % ((uint64_t)pb->D * mbs) != 0 || in->heads % tp != 0) return 0;      /* no valid plan in this problem */
    dp_ctx* c = (dp_ctx*)calloc(1, sizeof(dp_ctx));
    c->in = in; c->pb = pb; c->T = T; c->tp = tp; c->need = pb->D * tp;
    c->n_b = in->gbs / ((uint64_t)pb->D * mbs);
    c->msg = in->p2p_bytes[pb->mbs_idx];
    for (uint32_t i = 0; i < P; ++i)
        for (uint32_t g = 0; g < T; ++g) {
            uint64_t par;
            dp_stage(in, P, i, g, pb->tp_idx, pb->mbs_idx, pb->rc, c->n_b, &c->fb[i][g], &c->upd[i][g], &par, &c->fits[i][g]);
            c->params[i] = par;
        }
    dpb_val best; memset(&best, 0, sizeof(best));
    const uint8_t nothing[ORC_DP_T_MAX] = {0};
    for (uint32_t g = 0; g < T; ++g) {                       /* stage 0: every type, first fit from the first zone */
        const int zp = first_fit(c, 0, nothing, g);
        if (zp < 0) continue;
        uint8_t used[ORC_DP_T_MAX] = {0};
        used[g] = 1;
        const dpb_val v = solve_suffix_budget(c, 0, g, (uint32_t)zp, used, limit);
        if (!v.found) continue;
        if (!best.found || dpb_value(c, &v) < dpb_value(c, &best)) best = v;
    }
    out->n_states = c->n_states;
    if (best.found) {
        out->found = 1;
        out->value = dpb_value(c, &best);
        out->charged_cost = best.cost;
        orc_plan* pl = &out->plan;
        pl->P = P; pl->mbs_idx = pb->mbs_idx; pl->rc = pb->rc; pl->D = pb->D;
        uint8_t used[ORC_DP_T_MAX] = {0};
        uint32_t zp = 0;
        for (uint32_t i = 0; i < P; ++i) {                   /* zones by first fit, as the recursion placed them */
            const uint32_t g = best.type[i];
            const int zp2 = first_fit(c, zp, used, g);
            if ((uint32_t)zp2 != zp) memset(used, 0, sizeof(used));
            used[g]++;
            zp = (uint32_t)zp2;
            pl->type[i] = g; pl->zone[i] = pb->zone_list[zp]; pl->tp_idx[i] = pb->tp_idx;
        }
    }
    free(c);
    return 0;
}

/* ---- plans whose stages mix GPU types among their replicas (Sec. 4.2, Sec. 4.3, Sec. 4.4) -----------
 *
 * Stage i has D replicas in one zone (H5), given as groups: `count` replicas on one GPU type with one
 * tensor-parallel degree (H1).  Replicas are numbered group after group, and pipeline k runs on replica
 * k of every stage, so the pipelines differ and T_iter takes the slowest one (Sec. 4.3).
 */
void orc_simulate_mixed(const orc_inputs* in, const orc_mixed_plan* pl, orc_out* out) {
    static uint8_t kinds[ORC_STAGES_MAX][1024 + 2];
    uint32_t nl[ORC_STAGES_MAX];
    const uint32_t P = pl->P, T = in->n_types, Z = in->n_zones;
    const uint32_t mbs_idx = pl->mbs_idx, D = pl->D, rc = pl->rc;
    const uint64_t mbs = in->mbs_values[mbs_idx];
    uint32_t status = 0;
    memset(out, 0, sizeof(*out));

    /* validity: the batch divides evenly, every stage has exactly D replicas, tensor parallelism stays in a node */
    if (D == 0 || in->gbs % ((uint64_t)D * mbs) != 0) status |= ORC_INVALID;
    for (uint32_t i = 0; i < P; ++i) {
        uint64_t replicas = 0;
        for (uint32_t q = 0; q < pl->stage[i].n_groups; ++q) {
            const orc_replica_group* gr = &pl->stage[i].group[q];
            const uint32_t tp = in->tp_values[gr->tp_idx];
            replicas += gr->count;
            if (gr->count == 0 || tp > in->gpus_per_node[gr->type] || in->heads % tp != 0) status |= ORC_INVALID;
        }
        if (replicas != D) status |= ORC_INVALID;
    }
    const uint64_t n_b = D ? in->gbs / ((uint64_t)D * mbs) : 0;
    out->n_b = n_b;

    /* resources */
    uint64_t used[64 * 64];
    memset(used, 0, sizeof(uint64_t) * Z * T);
    for (uint32_t i = 0; i < P; ++i)
        for (uint32_t q = 0; q < pl->stage[i].n_groups; ++q) {
            const orc_replica_group* gr = &pl->stage[i].group[q];
            used[pl->stage[i].zone * T + gr->type] += (uint64_t)gr->count * in->tp_values[gr->tp_idx];
        }
    for (uint32_t d = 0; d < Z * T; ++d)
        if (used[d] > in->avail[d]) status |= ORC_OVER_AVAIL;

    /* memory of every kind of worker: M_peak = M_model + M_activation */
    uint64_t params_stage[ORC_STAGES_MAX];
    uint64_t peak = 0;
    for (uint32_t i = 0; i < P; ++i) {
        nl[i] = stage_layers(in, P, i, kinds[i]);
        uint64_t stage_peak = 0;
        for (uint32_t q = 0; q < pl->stage[i].n_groups; ++q) {
            const orc_replica_group* gr = &pl->stage[i].group[q];
            const uint32_t tpi = gr->tp_idx;
            const uint64_t tp = in->tp_values[tpi];
            uint64_t params = 0, A = 0, W = 0;
            for (uint32_t l = 0; l < nl[i]; ++l) {
                const uint32_t k = kinds[i][l];
                params += in->params[k];
                A += rc ? tab_act(in, in->act_ckpt, k, tpi, mbs_idx) : tab_act(in, in->act_saved, k, tpi, mbs_idx);
                const uint64_t w = rc ? tab_act(in, in->act_saved, k, tpi, mbs_idx) : tab_act(in, in->act_work, k, tpi, mbs_idx);
                if (w > W) W = w;
            }
            params_stage[i] = params;
            const uint64_t m = ceil_div_u64(params, tp) * in->mul_factor * in->dtype_size +
                               min_u64((uint64_t)(P - i), n_b) * A + W + in->reserved[gr->type];
            if (m > in->capacity[gr->type]) status |= ORC_OOM;
            if (m > stage_peak) stage_peak = m;
        }
        out->stage_mem[i] = stage_peak;
        if (stage_peak > peak) peak = stage_peak;
    }
    out->peak_mem = peak;
    out->status = status;
    if (status & ORC_INVALID) {
        out->t_iter = NAN;
        out->cost = NAN;
        return;
    }

    /* the pipelines, one after the other: pipeline k uses, in stage i, the group that holds replica k */
    const uint64_t msg = in->p2p_bytes[mbs_idx];
    double max_pp = 0.0;
    for (uint32_t k = 0; k < D; ++k) {
        uint32_t grp[ORC_STAGES_MAX];
        for (uint32_t i = 0; i < P; ++i) {
            uint32_t q = 0, upto = pl->stage[i].group[0].count;
            while (k >= upto) { ++q; upto += pl->stage[i].group[q].count; }
            grp[i] = q;
        }
        double sum_t = 0.0, max_t = 0.0;
        for (uint32_t i = 0; i < P; ++i) {
            const orc_replica_group* gr = &pl->stage[i].group[grp[i]];
            const uint32_t g = gr->type, z = pl->stage[i].zone, tpi = gr->tp_idx;
            double f = 0.0, b = 0.0;
            for (uint32_t l = 0; l < nl[i]; ++l) {
                f = f + tab4(in, in->fwd, kinds[i][l], g, tpi, mbs_idx);
                b = b + tab4(in, in->bwd, kinds[i][l], g, tpi, mbs_idx);
            }
            if (rc) b = b + f;
            double c = 0.0;
            if (i + 1 < P) {
                const orc_replica_group* g2r = &pl->stage[i + 1].group[grp[i + 1]];
                const uint32_t g2 = g2r->type, z2 = pl->stage[i + 1].zone;
                if (z != z2) {
                    c = link_time(in->zone_alpha[z * Z + z2], in->zone_inv_bw[z * Z + z2], poly_at(in->zone_bw_poly, z * Z + z2), msg);
                } else if (g == g2 && (uint64_t)gr->count * in->tp_values[tpi] + (uint64_t)g2r->count * in->tp_values[g2r->tp_idx] <=
                                          in->gpus_per_node[g]) {
                    /* the two groups' GPUs all sit in one node */
                    c = link_time(in->intra_alpha[z * T + g], in->intra_inv_bw[z * T + g], poly_at(in->intra_bw_poly, z * T + g), msg);
                } else {
                    const double c1 = link_time(in->inter_alpha[z * T + g], in->inter_inv_bw[z * T + g], poly_at(in->inter_bw_poly, z * T + g), msg);
                    const double c2 = link_time(in->inter_alpha[z * T + g2], in->inter_inv_bw[z * T + g2], poly_at(in->inter_bw_poly, z * T + g2), msg);
                    c = max_f64(c1, c2);
                }
            }
            const double t = (f + b) + 2.0 * c;
            sum_t = sum_t + t;
            max_t = max_f64(max_t, t);
        }
        const double t_pp = sum_t + (double)n_b * max_t;
        max_pp = max_f64(max_pp, t_pp);
    }

    /* synchronisation and update: the slowest over stages, and within a stage over its groups */
    double max_sync = 0.0, max_u = 0.0;
    for (uint32_t i = 0; i < P; ++i) {
        const uint32_t z = pl->stage[i].zone, ng = pl->stage[i].n_groups;
        /* the ring moves the largest shard (the group with the smallest tp sets the message size) */
        uint64_t gradbytes = 0;
        for (uint32_t q = 0; q < ng; ++q) {
            const uint64_t gb = ceil_div_u64(params_stage[i], in->tp_values[pl->stage[i].group[q].tp_idx]) * in->grad_dtype_size;
            if (gb > gradbytes) gradbytes = gb;
        }
        double sync = 0.0;
        for (uint32_t q = 0; q < ng; ++q) {
            const orc_replica_group* gr = &pl->stage[i].group[q];
            const uint32_t g = gr->type, d = z * T + g;
            double u = 0.0;
            for (uint32_t l = 0; l < nl[i]; ++l) u = u + tab_upd(in, kinds[i][l], g, gr->tp_idx);
            max_u = max_f64(max_u, u);
            if (D > 1) {
                /* one group whose GPUs fit a node talks inside the node; otherwise every group's inter-node
                 * link carries the ring and the slowest of them sets the time */
                const int intra = ng == 1 && (uint64_t)D * in->tp_values[gr->tp_idx] <= in->gpus_per_node[g];
                const double alpha = intra ? in->intra_alpha[d] : in->inter_alpha[d];
                const double inv = intra ? in->intra_inv_bw[d] : in->inter_inv_bw[d];
                const double* poly = intra ? poly_at(in->intra_bw_poly, d) : poly_at(in->inter_bw_poly, d);
                const double steps = (double)(2 * (uint64_t)(D - 1));
                const double coef = steps / (double)D;
                double s;
                if (poly) s = (coef * (double)gradbytes) / poly_bw(poly, (double)gradbytes / (double)D) + steps * alpha;
                else s = (coef * (double)gradbytes) * inv + steps * alpha;
                sync = max_f64(sync, s);
            }
        }
        out->stage_sync[i] = sync;
        max_sync = max_f64(max_sync, sync);
    }
    const double t_iter = (max_pp + max_sync) + max_u;
    out->t_pp = max_pp;
    out->t_sync = max_sync;
    out->t_update = max_u;
    out->t_iter = t_iter;

    /* cost: every replica's GPUs for the whole iteration, and the bytes that cross zones */
    double rate = 0.0;
    for (uint32_t i = 0; i < P; ++i)
        for (uint32_t q = 0; q < pl->stage[i].n_groups; ++q) {
            const orc_replica_group* gr = &pl->stage[i].group[q];
            const uint32_t n_gpus = gr->count * in->tp_values[gr->tp_idx];
            rate = rate + (double)n_gpus * (in->price_per_hour[pl->stage[i].zone * T + gr->type] / 3600.0);
        }
    double c_comm = 0.0;
    for (uint32_t i = 0; i + 1 < P; ++i) {
        const uint32_t z = pl->stage[i].zone, z2 = pl->stage[i + 1].zone;
        if (z != z2) c_comm = c_comm + (double)(2 * n_b * (uint64_t)D * msg) * in->egress[z * Z + z2];
    }
    out->rate_per_s = rate;
    out->c_comm = c_comm;
    out->cost = rate * t_iter + c_comm;
}

void orc_simulate_mixed_batch(const orc_inputs* in, const orc_mixed_plan* plans, uint64_t n, uint32_t* status,
                              double* t_iter, double* cost, uint64_t* peak_mem) {
    orc_out o;
    for (uint64_t j = 0; j < n; ++j) {
        orc_simulate_mixed(in, &plans[j], &o);
        status[j] = o.status;
        t_iter[j] = o.t_iter;
        cost[j] = o.cost;
        peak_mem[j] = o.peak_mem;
    }
}

/* ---- searching over plans with mixed replicas (Sec. 4.2.2, "Implementation") ----------------------------- */

static uint32_t mixed_units(const orc_mixed_space* sp, uint32_t D) {
    return (sp->granularity >= 1 && D % sp->granularity == 0) ? sp->granularity : D;
}

/* Walks the combinations in DESCENDING lexicographic order (all replicas on type 0 comes first, so that with one unit
 * combination c is "everything on type c"), plainly: type 0's units from the most down, inside that type 1's, and so
 * on, the last type taking what is left; tuples with more than ORC_GROUPS_MAX non-zero entries are skipped.
 * Returns how many there are; the tuple of index `want` is left in `u`. */
static uint64_t walk_combs(uint32_t T, uint32_t units, uint64_t want, uint32_t* u, int* found) {
    uint64_t n = 0;
    uint32_t cur[ORC_DP_T_MAX];
    for (uint32_t t = 0; t < ORC_DP_T_MAX; ++t) cur[t] = units;
    for (;;) {
        uint32_t used = 0, nonzero = 0;
        for (uint32_t t = 0; t + 1 < T; ++t) { used += cur[t]; nonzero += cur[t] != 0; }
        if (used <= units) {
            const uint32_t last = units - used;
            if (nonzero + (last != 0) <= ORC_GROUPS_MAX) {
                if (n == want && u) {
                    for (uint32_t t = 0; t + 1 < T; ++t) u[t] = cur[t];
                    u[T - 1] = last;
                    if (found) *found = 1;
                }
                n++;
            }
        }
        /* previous tuple of the first T - 1 entries in lexicographic order: the last of them fastest */
        int t = (int)T - 2;
        while (t >= 0 && cur[t] == 0) { cur[t] = units; t--; }
        if (t < 0) break;
        cur[t]--;
    }
    return n;
}

uint64_t orc_mixed_n_comb(const orc_inputs* in, const orc_mixed_space* sp, uint32_t D) {
    return walk_combs(in->n_types, mixed_units(sp, D), ~0ull, NULL, NULL);
}

int orc_mixed_comb(const orc_inputs* in, const orc_mixed_space* sp, uint32_t D, uint64_t c, uint32_t* units_per_type) {
    int found = 0;
    walk_combs(in->n_types, mixed_units(sp, D), c, units_per_type, &found);
    return found ? 0 : -1;
}

static uint32_t mixed_nseg(const orc_mixed_space* sp, uint32_t P) { return P < sp->seg_max ? P : sp->seg_max; }

uint64_t orc_mixed_space_size(const orc_inputs* in, const orc_mixed_space* sp) {
    uint64_t n = 0;
    for (uint32_t jp = 0; jp < sp->n_p; ++jp)
        for (uint32_t jd = 0; jd < sp->n_d; ++jd) {
            const uint64_t radix = (uint64_t)in->n_zones * orc_mixed_n_comb(in, sp, sp->d_values[jd]);
            n += (uint64_t)sp->n_mbs * sp->n_rc * ipow_u64(radix, mixed_nseg(sp, sp->p_values[jp]));
        }
    return n;
}

int orc_mixed_decode(const orc_inputs* in, const orc_mixed_space* sp, uint64_t flat, orc_mixed_plan* out) {
    memset(out, 0, sizeof(*out));
    for (uint32_t jp = 0; jp < sp->n_p; ++jp) {
        const uint32_t P = sp->p_values[jp], nseg = mixed_nseg(sp, P);
        for (uint32_t mi = 0; mi < sp->n_mbs; ++mi)
        for (uint32_t ri = 0; ri < sp->n_rc; ++ri)
        for (uint32_t jd = 0; jd < sp->n_d; ++jd) {
            const uint32_t D = sp->d_values[jd];
            const uint64_t n_comb = orc_mixed_n_comb(in, sp, D), radix = (uint64_t)in->n_zones * n_comb;
            const uint64_t block = ipow_u64(radix, nseg);
            if (flat >= block) { flat -= block; continue; }
            uint64_t digit[ORC_STAGES_MAX];
            for (uint32_t s = nseg; s-- > 0;) { digit[s] = flat % radix; flat /= radix; }
            out->P = P; out->mbs_idx = sp->mbs_idx[mi]; out->rc = sp->rc_values[ri]; out->D = D;
            const uint32_t units = mixed_units(sp, D), per_unit = D / units;
            uint32_t u[ORC_GROUPS_MAX][ORC_DP_T_MAX];        /* the combination of each segment (nseg <= seg_max <= 4) */
            if (nseg > ORC_GROUPS_MAX) return -1;
            for (uint32_t s = 0; s < nseg; ++s)
                if (orc_mixed_comb(in, sp, D, digit[s] % n_comb, u[s]) != 0) return -1;
            for (uint32_t i = 0; i < P; ++i) {
                const uint32_t sg = (uint32_t)((uint64_t)i * nseg / P);
                orc_mixed_stage* st = &out->stage[i];
                st->zone = (uint32_t)(digit[sg] / n_comb);
                st->n_groups = 0;
                for (uint32_t g = 0; g < in->n_types; ++g) {
                    if (!u[sg][g]) continue;
                    st->group[st->n_groups].type = g;
                    st->group[st->n_groups].tp_idx = sp->tp_idx_of_type[g];
                    st->group[st->n_groups].count = u[sg][g] * per_unit;
                    st->n_groups++;
                }
            }
            return 0;
        }
    }
    return -1;
}

uint32_t orc_search_mixed(const orc_inputs* in, const orc_mixed_space* sp, const orc_objective* obj, uint64_t lo,
                          uint64_t hi, uint32_t k, orc_hit* hits, orc_counts* counts) {
    static orc_mixed_plan pl;
    orc_out o;
    uint32_t n_hits = 0;
    orc_counts c;
    memset(&c, 0, sizeof(c));
    for (uint64_t flat = lo; flat < hi; ++flat) {
        if (orc_mixed_decode(in, sp, flat, &pl) != 0) break;
        orc_simulate_mixed(in, &pl, &o);
        c.n_total++;
        if (o.status & ORC_INVALID) { c.n_invalid++; continue; }
        if (o.status & ORC_OOM) { c.n_oom++; continue; }
        if (o.status & ORC_OVER_AVAIL) { c.n_over_avail++; continue; }
        int over = 0;
        if (obj->budget > 0.0 && o.cost > obj->budget) over = 1;
        if (obj->min_rate > 0.0 && 1.0 / o.t_iter < obj->min_rate) over = 1;
        if (over) { c.n_over_constraint++; continue; }
        c.n_feasible++;
        if (c.n_feasible == 1 || o.cost < c.min_cost) c.min_cost = o.cost;
        n_hits = offer_hit(hits, n_hits, k, flat, score_of(obj, &o), &o);
    }
    if (counts) *counts = c;
    return n_hits;
}
