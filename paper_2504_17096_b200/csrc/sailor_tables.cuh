// Device-side table layout, flat-index decoding and the per-record simulator.
//
// All tables of one context live in one contiguous device "blob": a fixed header followed
// by the variable-size arrays at 16-byte aligned offsets.  The part up to `static_bytes`
// (header + raw profile + cluster tables, a few KB) is what kernels stage in shared
// memory; the left-to-right layer-sum chains are larger and stay in global memory (L2).
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/sailor.h"

namespace sailor {

constexpr int KIND_EMBED = 0, KIND_BLOCK = 1, KIND_HEAD = 2;
constexpr int R_MAX = SAILOR_T_MAX * SAILOR_Z_MAX;   // digits: zone * T + type

struct alignas(16) TabHdr {
    // model
    uint32_t n_blocks, has_embed, has_head, heads;
    uint64_t gbs;
    uint64_t mul_bytes;        // mul_factor * dtype_size, bytes per parameter on a worker
    uint64_t grad_bytes;       // bytes per gradient element
    // shapes
    uint32_t T, Z, R, n_tp, n_mbs, chain_len;   // chain_len = n_blocks + 1
    uint32_t tp_values[SAILOR_TP_MAX];
    uint32_t mbs_values[SAILOR_MBS_MAX];
    uint32_t gpn[SAILOR_T_MAX];
    uint64_t capacity[SAILOR_T_MAX];
    uint64_t reserved[SAILOR_T_MAX];
    uint64_t params[SAILOR_KINDS];
    // byte offsets from the blob start
    uint32_t off_fwd, off_bwd, off_upd;           // f64 [kind][type][tp][mbs], [kind][type][tp]
    uint32_t off_saved, off_ckpt, off_work;       // u64 [kind][tp][mbs]
    uint32_t off_p2p;                             // u64 [mbs]
    uint32_t off_price_s;                         // f64 [digit]  price_per_hour / 3600
    uint32_t off_intra_a, off_intra_i, off_inter_a, off_inter_i;   // f64 [digit]
    uint32_t off_zone_a, off_zone_i, off_egress;  // f64 [zone][zone]
    uint32_t off_intra_p, off_inter_p, off_zone_p; // f64 [..][4] bandwidth polynomials, 0 = none
    uint32_t static_bytes;                        // multiple of 16
    uint32_t off_chain_f, off_chain_b;            // f64 [start][type][tp][mbs][chain_len]
    uint32_t off_chain_u;                         // f64 [start][type][tp][chain_len]
    uint32_t total_bytes;
    // per stage composition c = (embedding * 2 + head) * chain_len + blocks: what a stage of that make-up needs,
    // formed once per context so that a simulated stage is a handful of loads
    uint32_t off_cmp_params;                      // u64 [c]                        parameters
    uint32_t off_cmp_grad;                        // f64 [c][tp]                    gradient bytes of one worker, as a double
    uint32_t off_cmp_mem;                         // u64 [c][tp][mbs][rc][2]        model + working bytes, bytes kept per in-flight microbatch
    uint32_t off_cmp_fb;                          // f64 [c][type][tp][mbs][rc]     f + b (+ f with recomputation)
    uint32_t off_cmp_upd;                         // f64 [c][type][tp]              update time
    // tables of the explicit-batch kernel (sailor_batch.cuh)
    uint32_t off_piece;                           // PieceRec [c][type][tp][mbs][rc]
    uint32_t off_lnk_intra2, off_lnk_inter2;      // f64 [digit][mbs]   2 x one-way message time of the link
    uint32_t off_lnk_zone2;                       // f64 [zone][zone][mbs]
    uint32_t heads_ok;                            // bit i: tp_values[i] divides the number of attention heads
    uint32_t _pad[2];
};
static_assert(sizeof(TabHdr) % 16 == 0, "header must keep the arrays 16-byte aligned");

// Typed view over a blob whose static part may sit in shared memory and whose chains sit in
// global memory.
struct TabView {
    const TabHdr* h;
    const double *fwd, *bwd, *upd;
    const uint64_t *saved, *ckpt, *work, *p2p;
    const double *price_s, *intra_a, *intra_i, *inter_a, *inter_i, *zone_a, *zone_i, *egress;
    const double *intra_p, *inter_p, *zone_p;      // nullptr when the link class has no polynomial
    const double *chain_f, *chain_b, *chain_u;
    const uint64_t *cmp_params, *cmp_mem;
    const double *cmp_grad, *cmp_fb, *cmp_upd;

    __host__ __device__ void bind(const unsigned char* stat, const unsigned char* glob) {
        h = reinterpret_cast<const TabHdr*>(stat);
        fwd = reinterpret_cast<const double*>(stat + h->off_fwd);
        bwd = reinterpret_cast<const double*>(stat + h->off_bwd);
        upd = reinterpret_cast<const double*>(stat + h->off_upd);
        saved = reinterpret_cast<const uint64_t*>(stat + h->off_saved);
        ckpt = reinterpret_cast<const uint64_t*>(stat + h->off_ckpt);
        work = reinterpret_cast<const uint64_t*>(stat + h->off_work);
        p2p = reinterpret_cast<const uint64_t*>(stat + h->off_p2p);
        price_s = reinterpret_cast<const double*>(stat + h->off_price_s);
        intra_a = reinterpret_cast<const double*>(stat + h->off_intra_a);
        intra_i = reinterpret_cast<const double*>(stat + h->off_intra_i);
        inter_a = reinterpret_cast<const double*>(stat + h->off_inter_a);
        inter_i = reinterpret_cast<const double*>(stat + h->off_inter_i);
        zone_a = reinterpret_cast<const double*>(stat + h->off_zone_a);
        zone_i = reinterpret_cast<const double*>(stat + h->off_zone_i);
        egress = reinterpret_cast<const double*>(stat + h->off_egress);
        intra_p = h->off_intra_p ? reinterpret_cast<const double*>(stat + h->off_intra_p) : nullptr;
        inter_p = h->off_inter_p ? reinterpret_cast<const double*>(stat + h->off_inter_p) : nullptr;
        zone_p = h->off_zone_p ? reinterpret_cast<const double*>(stat + h->off_zone_p) : nullptr;
        chain_f = reinterpret_cast<const double*>(glob + h->off_chain_f);
        chain_b = reinterpret_cast<const double*>(glob + h->off_chain_b);
        chain_u = reinterpret_cast<const double*>(glob + h->off_chain_u);
        cmp_params = reinterpret_cast<const uint64_t*>(glob + h->off_cmp_params);
        cmp_grad = reinterpret_cast<const double*>(glob + h->off_cmp_grad);
        cmp_mem = reinterpret_cast<const uint64_t*>(glob + h->off_cmp_mem);
        cmp_fb = reinterpret_cast<const double*>(glob + h->off_cmp_fb);
        cmp_upd = reinterpret_cast<const double*>(glob + h->off_cmp_upd);
    }
};

// ---- arithmetic helpers: one rounding per operation, never contracted ---------------------
__device__ __forceinline__ double add_rn(double a, double b) { return __dadd_rn(a, b); }
__device__ __forceinline__ double mul_rn(double a, double b) { return __dmul_rn(a, b); }
__host__ __device__ __forceinline__ double dmax(double a, double b) { return a > b ? a : b; }

// Forward / backward / update time of one stage on (type g, tp index, mbs index): the
// left-to-right sum over [embed?] + nb blocks + [head?], read from the chain tables.
struct StageTimes { double f, b, u; };

__device__ __forceinline__ StageTimes stage_times(const TabView& v, uint32_t g, uint32_t tpi, uint32_t mi,
                                                  uint32_t nb, bool e, bool hd) {
    const TabHdr* h = v.h;
    const uint32_t gt = (g * h->n_tp + tpi);
    const size_t tstride = (size_t)h->T * h->n_tp;
    const size_t i3 = (size_t)(e ? tstride : 0) + gt;
    const size_t i4 = i3 * h->n_mbs + mi;
    StageTimes s;
    s.f = v.chain_f[i4 * h->chain_len + nb];
    s.b = v.chain_b[i4 * h->chain_len + nb];
    s.u = v.chain_u[i3 * h->chain_len + nb];
    if (hd) {
        const size_t k4 = (((size_t)KIND_HEAD * h->T + g) * h->n_tp + tpi);
        s.f = add_rn(s.f, v.fwd[k4 * h->n_mbs + mi]);
        s.b = add_rn(s.b, v.bwd[k4 * h->n_mbs + mi]);
        s.u = add_rn(s.u, v.upd[k4]);
    }
    return s;
}

// ceil(a / b) for b >= 1; tensor-parallel degrees are powers of two in practice, which avoids the
// 64-bit division routine.
__host__ __device__ __forceinline__ uint64_t ceil_div64(uint64_t a, uint32_t b) {
    if ((b & (b - 1u)) == 0u) {
#ifdef __CUDA_ARCH__
        return (a + b - 1u) >> (31 - __clz((int)b));
#else
        uint32_t sh = 0;
        while ((1u << sh) < b) ++sh;
        return (a + b - 1u) >> sh;
#endif
    }
    return (a + b - 1u) / b;
}

// Parameters of stage i and its per-worker peak memory without the reserved bytes
// (Sec. 4.3: M_peak = M_model + M_activation; stage i keeps min(P - i, N_b) microbatches).
struct StageMem { uint64_t params, mem; };

__device__ __forceinline__ StageMem stage_memory(const TabView& v, uint32_t tpi, uint32_t mi, uint32_t rc,
                                                 uint32_t nb, bool e, bool hd, uint64_t inflight) {
    const TabHdr* h = v.h;
    const uint32_t tp = h->tp_values[tpi];
    auto at = [&](const uint64_t* t, int kind) { return t[((size_t)kind * h->n_tp + tpi) * h->n_mbs + mi]; };
    const uint64_t* keep = rc ? v.ckpt : v.saved;
    const uint64_t* wset = rc ? v.saved : v.work;
    uint64_t params = (uint64_t)nb * h->params[KIND_BLOCK];
    uint64_t A = (uint64_t)nb * at(keep, KIND_BLOCK);
    uint64_t W = nb ? at(wset, KIND_BLOCK) : 0;
    if (e) {
        params += h->params[KIND_EMBED];
        A += at(keep, KIND_EMBED);
        const uint64_t w = at(wset, KIND_EMBED);
        W = w > W ? w : W;
    }
    if (hd) {
        params += h->params[KIND_HEAD];
        A += at(keep, KIND_HEAD);
        const uint64_t w = at(wset, KIND_HEAD);
        W = w > W ? w : W;
    }
    StageMem m;
    m.params = params;
    m.mem = ceil_div64(params, tp) * h->mul_bytes + inflight * A + W;
    return m;
}

// Bandwidth of a link for a message of m bytes from its fitted polynomial (Sec. 4.1), Horner form.
__device__ __forceinline__ double poly_bw(const double* p, double m) {
    return add_rn(mul_rn(add_rn(mul_rn(add_rn(mul_rn(p[3], m), p[2]), m), p[1]), m), p[0]);
}
// Time of a message of m bytes: alpha + m / bandwidth(m) with a polynomial, else alpha + m * inv_bw.
__device__ __forceinline__ double link_time(double alpha, double inv_bw, const double* table, uint32_t idx, double m) {
    if (table) return add_rn(alpha, m / poly_bw(table + 4 * idx, m));
    return add_rn(alpha, mul_rn(m, inv_bw));
}

// Time of one message over the link between neighbouring stages (one direction).
__device__ __forceinline__ double boundary_time(const TabView& v, uint32_t g, uint32_t z, uint32_t tp,
                                                uint32_t g2, uint32_t z2, uint32_t tp2, uint32_t D, double msg) {
    const TabHdr* h = v.h;
    if (z != z2) return link_time(v.zone_a[z * h->Z + z2], v.zone_i[z * h->Z + z2], v.zone_p, z * h->Z + z2, msg);
    const uint32_t d = z * h->T + g;
    if (g == g2 && (uint64_t)D * (tp + tp2) <= h->gpn[g]) return link_time(v.intra_a[d], v.intra_i[d], v.intra_p, d, msg);
    const uint32_t d2 = z * h->T + g2;
    const double c1 = link_time(v.inter_a[d], v.inter_i[d], v.inter_p, d, msg);
    const double c2 = link_time(v.inter_a[d2], v.inter_i[d2], v.inter_p, d2, msg);
    return dmax(c1, c2);
}

// Ring all-reduce of `params` parameters' gradients (split over tp) among D replicas on the link of
// digit d (H5: inside one zone): 2(D-1) messages of gradbytes / D.
__device__ __forceinline__ double allreduce_time(const TabView& v, uint32_t g, uint32_t d, uint32_t tp, uint32_t D,
                                                 uint64_t params, double steps, double coef) {
    const TabHdr* h = v.h;
    const bool intra = (uint64_t)D * tp <= h->gpn[g];
    const double alpha = intra ? v.intra_a[d] : v.inter_a[d];
    const double* poly = intra ? v.intra_p : v.inter_p;
    const double gradbytes = (double)(ceil_div64(params, tp) * h->grad_bytes);
    const double volume = mul_rn(coef, gradbytes);
    double t;
    if (poly) t = volume / poly_bw(poly + 4 * d, gradbytes / (double)D);
    else t = mul_rn(volume, intra ? v.intra_i[d] : v.inter_i[d]);
    return add_rn(t, mul_rn(steps, alpha));
}

// The same ring with the gradient bytes of one worker given (as a double) and the link class decided by the caller.
__device__ __forceinline__ double allreduce_bytes_time(const TabView& v, uint32_t d, bool intra, double gradbytes, uint32_t D,
                                                       double steps, double coef) {
    const double alpha = intra ? v.intra_a[d] : v.inter_a[d];
    const double* poly = intra ? v.intra_p : v.inter_p;
    const double volume = mul_rn(coef, gradbytes);
    double t;
    if (poly) t = volume / poly_bw(poly + 4 * d, gradbytes / (double)D);
    else t = mul_rn(volume, intra ? v.intra_i[d] : v.inter_i[d]);
    return add_rn(t, mul_rn(steps, alpha));
}

__device__ __forceinline__ double sync_time(const TabView& v, uint32_t g, uint32_t z, uint32_t tp, uint32_t D,
                                            uint64_t params) {
    if (D <= 1) return 0.0;
    const double steps = (double)(2 * (uint64_t)(D - 1));
    return allreduce_time(v, g, z * v.h->T + g, tp, D, params, steps, steps / (double)D);
}

struct SimOut {
    double t_iter, cost;
    uint64_t peak_mem;
    uint32_t status;
};

__device__ __forceinline__ double make_nan() { return __longlong_as_double(0x7ff8000000000000LL); }
__device__ __forceinline__ double make_inf() { return __longlong_as_double(0x7ff0000000000000LL); }

// Simulate one run-length encoded plan (Sec. 4.3), given as its header values and `n_runs` runs
// (at most `max_runs`).  Every index is checked before use; a plan that fails gets
// SAILOR_ST_BAD_RECORD and nothing is read through it.
//
// The stages are walked in one flat loop (no loop nest over runs), so that the lanes of a warp,
// each with its own record, stay on the same instructions; values that depend only on the
// stage's layer composition and run are refreshed when either changes.  `cnt` points to this
// thread's per-digit GPU counters (digit d at cnt[d * cnt_stride], any initial contents).
__device__ __forceinline__ SimOut simulate_runs(const TabView& v, const uint16_t* __restrict__ avail, uint32_t P,
                                                uint32_t n_runs, uint32_t D, uint32_t mi, uint32_t rc,
                                                const sailor_run* runs, uint32_t max_runs, uint32_t* cnt,
                                                uint32_t cnt_stride) {
    const TabHdr* h = v.h;
    SimOut o;
    o.t_iter = o.cost = make_nan();
    o.peak_mem = 0;
    o.status = SAILOR_ST_BAD_RECORD;
    if (P < 1 || P > SAILOR_P_MAX || n_runs < 1 || n_runs > max_runs || D < 1 || mi >= h->n_mbs) return o;
    uint32_t tot = 0;
    for (uint32_t q = 0; q < n_runs; ++q) {
        const sailor_run rr = runs[q];
        if (rr.type >= h->T || rr.zone >= h->Z || rr.tp_idx >= h->n_tp || rr.n_stages < 1) return o;
        tot += rr.n_stages;
    }
    if (tot != P) return o;

    uint32_t status = 0;
    const uint64_t mbs = h->mbs_values[mi];
    const uint64_t dm = (uint64_t)D * mbs;
    uint64_t n_b;
    if (((h->gbs | dm) >> 32) == 0) {                      // the usual case: a 32-bit division
        const uint32_t q32 = (uint32_t)h->gbs / (uint32_t)dm;
        n_b = q32;
        if (q32 * (uint32_t)dm != (uint32_t)h->gbs) status |= SAILOR_ST_INVALID;
    } else {
        n_b = h->gbs / dm;
        if (n_b * dm != h->gbs) status |= SAILOR_ST_INVALID;
    }

    // resources: GPUs taken of every (zone, type) the plan uses, saturating at 2^32 - 1 (availability is 16 bits)
    for (uint32_t q = 0; q < n_runs; ++q) cnt[(runs[q].zone * h->T + runs[q].type) * cnt_stride] = 0;
    for (uint32_t q = 0; q < n_runs; ++q) {
        const sailor_run a = runs[q];
        const uint32_t tp = h->tp_values[a.tp_idx];
        if (tp > h->gpn[a.type] || h->heads % tp != 0) status |= SAILOR_ST_INVALID;
        uint32_t* c = cnt + (a.zone * h->T + a.type) * cnt_stride;
        const uint64_t sum = (uint64_t)*c + (uint64_t)D * tp * a.n_stages;
        *c = sum > 0xffffffffull ? 0xffffffffu : (uint32_t)sum;
    }
    for (uint32_t q = 0; q < n_runs; ++q) {
        const uint32_t d = runs[q].zone * h->T + runs[q].type;
        if (cnt[d * cnt_stride] > avail[d]) status |= SAILOR_ST_OVER_AVAIL;
    }

    const uint32_t base = h->n_blocks / P, extra = h->n_blocks % P;
    const double msg = (double)v.p2p[mi];
    const uint64_t xbytes = 2 * n_b * (uint64_t)D * v.p2p[mi];
    const double steps = (double)(2 * (uint64_t)(D - 1));
    const double coef = steps / (double)D;                 // ring all-reduce: 2(D-1)/D
    double sum_t = 0.0, max_t = 0.0, max_sync = 0.0, max_u = 0.0, rate = 0.0, c_comm = 0.0;
    uint64_t peak = 0;

    // The stages are walked piece by piece: a piece is a stretch of one run with one layer make-up, so all its
    // stages have the same f + b, memory terms and synchronisation; only the stage that closes a run (it sends to
    // the next run) and the final stage (it sends nothing) have a time of their own.  Within a piece the sums take
    // one addition per stage, in stage order, exactly as a stage-by-stage walk would add them; memory is largest at
    // the piece's first stage (the in-flight microbatches never grow with the stage index), so that one is checked.
    uint32_t i = 0;
    for (uint32_t q = 0; q < n_runs; ++q) {
        const sailor_run a = runs[q];
        const uint32_t g = a.type, z = a.zone, tpi = a.tp_idx, tp = h->tp_values[tpi];
        const uint32_t d = z * h->T + g, run_end = i + a.n_stages;
        const double gpu_rate = mul_rn((double)(D * tp), v.price_s[d]);
        const uint64_t cap = h->capacity[g], resv = h->reserved[g];
        const double c2_self = mul_rn(2.0, boundary_time(v, g, z, tp, g, z, tp, D, msg));
        const bool intra_dp = (uint64_t)D * tp <= h->gpn[g];
        while (i < run_end) {
            const uint32_t nb = base + (i < extra ? 1u : 0u);
            const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
            // the piece ends with the run, after the embedding stage, where the extra blocks run out, before the head stage
            uint32_t piece_end = run_end;
            if (e) piece_end = 1;
            else {
                if (i < extra && extra < piece_end) piece_end = extra;
                if (h->has_head && i < P - 1 && P - 1 < piece_end) piece_end = P - 1;
            }
            // everything a stage of this make-up needs was formed once per context (compose_kernel)
            const size_t comp = (size_t)((e ? 2u : 0u) + (hd ? 1u : 0u)) * h->chain_len + nb;
            const size_t ct = comp * h->n_tp + tpi;
            const double fb = v.cmp_fb[(((comp * h->T + g) * h->n_tp + tpi) * h->n_mbs + mi) * 2 + rc];
            const double upd = v.cmp_upd[(comp * h->T + g) * h->n_tp + tpi];
            const uint64_t* mm = v.cmp_mem + ((ct * h->n_mbs + mi) * 2 + rc) * 2;
            const double sync = D > 1 ? allreduce_bytes_time(v, d, intra_dp, v.cmp_grad[ct], D, steps, coef) : 0.0;
            const uint64_t inflight = (uint64_t)(P - i) < n_b ? (uint64_t)(P - i) : n_b;
            const uint64_t m = mm[0] + resv + inflight * mm[1];
            if (m > cap) status |= SAILOR_ST_OOM;
            peak = m > peak ? m : peak;
            max_u = dmax(max_u, upd);
            max_sync = dmax(max_sync, sync);
            // stages of the piece whose receiver sits in the same run
            const bool closes = piece_end == run_end || piece_end == P;      // its last stage has a time of its own
            const uint32_t n_plain = piece_end - i - (closes ? 1u : 0u);
            if (n_plain) {
                const double t_self = add_rn(fb, c2_self);
                max_t = dmax(max_t, t_self);
                for (uint32_t n = 0; n < n_plain; ++n) {
                    sum_t = add_rn(sum_t, t_self);
                    rate = add_rn(rate, gpu_rate);
                }
            }
            if (closes) {
                double t = fb;                                       // the final stage sends nothing: fb + 2*0
                if (piece_end < P) {                                 // the next stage opens run q + 1
                    const sailor_run nx = runs[q + 1];
                    const double c = boundary_time(v, g, z, tp, nx.type, nx.zone, h->tp_values[nx.tp_idx], D, msg);
                    if (nx.zone != z) c_comm = add_rn(c_comm, mul_rn((double)xbytes, v.egress[z * h->Z + nx.zone]));
                    t = add_rn(fb, mul_rn(2.0, c));
                }
                sum_t = add_rn(sum_t, t);
                max_t = dmax(max_t, t);
                rate = add_rn(rate, gpu_rate);
            }
            i = piece_end;
        }
    }
    o.peak_mem = peak;
    o.status = status;
    if (status & SAILOR_ST_INVALID) return o;
    const double t_pp = add_rn(sum_t, mul_rn((double)n_b, max_t));
    o.t_iter = add_rn(add_rn(t_pp, max_sync), max_u);
    o.cost = add_rn(mul_rn(rate, o.t_iter), c_comm);
    return o;
}

__device__ inline SimOut simulate_record(const TabView& v, const uint16_t* __restrict__ avail,
                                         const sailor_plan_rec& r, uint32_t* cnt, uint32_t cnt_stride) {
    return simulate_runs(v, avail, r.P, r.n_runs, r.D, r.mbs_idx, r.rc ? 1u : 0u, r.run, SAILOR_RUN_MAX, cnt, cnt_stride);
}

// ---- search space -------------------------------------------------------------------------
struct SpaceDesc {
    uint32_t n_p, n_mbs, n_tp, n_rc, n_d, seg_max;
    uint8_t p_values[SAILOR_NP_MAX];
    uint8_t mbs_idx[SAILOR_MBS_MAX];
    uint8_t tp_idx[SAILOR_TP_MAX];
    uint8_t rc_values[2];
    uint16_t d_values[SAILOR_ND_MAX];
};

__host__ __device__ inline uint32_t nseg_of(uint32_t P, uint32_t seg_max) { return P < seg_max ? P : seg_max; }
__host__ __device__ inline uint64_t ipow64(uint64_t b, uint32_t e) {
    uint64_t r = 1;
    while (e--) r *= b;
    return r;
}

// One configuration = (P, mbs, tp, rc, D); index c counts them in enumeration order.
struct Config {
    uint32_t P, mi, tpi, rc, D, nseg;
};
__host__ __device__ inline Config config_of(const SpaceDesc& s, uint32_t c) {
    Config k;
    uint32_t x = c;
    const uint32_t di = x % s.n_d;  x /= s.n_d;
    const uint32_t ri = x % s.n_rc; x /= s.n_rc;
    const uint32_t ti = x % s.n_tp; x /= s.n_tp;
    const uint32_t mi = x % s.n_mbs; x /= s.n_mbs;
    k.P = s.p_values[x];
    k.mi = s.mbs_idx[mi];
    k.tpi = s.tp_idx[ti];
    k.rc = s.rc_values[ri];
    k.D = s.d_values[di];
    k.nseg = nseg_of(k.P, s.seg_max);
    return k;
}

// Flat index -> record.  Runs are the segments (equal neighbours are not merged, so that a
// record maps back to exactly one flat index).
__host__ __device__ inline bool decode_flat(const SpaceDesc& s, uint32_t T, uint32_t Z, uint64_t flat,
                                            sailor_plan_rec* out) {
    const uint64_t R = (uint64_t)T * Z;
    const uint64_t base = (uint64_t)s.n_mbs * s.n_tp * s.n_rc * s.n_d;
    for (uint32_t j = 0; j < s.n_p; ++j) {
        const uint32_t P = s.p_values[j];
        const uint32_t nseg = nseg_of(P, s.seg_max);
        const uint64_t sub = base * ipow64(R, nseg);
        if (flat >= sub) { flat -= sub; continue; }
        uint32_t seg[SAILOR_SEG_MAX];
        for (uint32_t q = nseg; q-- > 0;) { seg[q] = (uint32_t)(flat % R); flat /= R; }
        const uint32_t c = j * (uint32_t)base + (uint32_t)flat;
        const Config k = config_of(s, c);
        for (int q = 0; q < (int)sizeof(*out); ++q) reinterpret_cast<unsigned char*>(out)[q] = 0;
        out->P = (uint8_t)P;
        out->mbs_idx = (uint8_t)k.mi;
        out->rc = (uint8_t)k.rc;
        out->D = (uint16_t)k.D;
        out->n_runs = (uint8_t)nseg;
        for (uint32_t q = 0; q < nseg; ++q) {
            // stages of segment q: floor(i*nseg/P) == q  <=>  ceil(q*P/nseg) <= i < ceil((q+1)*P/nseg)
            const uint32_t a = (q * P + nseg - 1) / nseg, e = ((q + 1) * P + nseg - 1) / nseg;
            out->run[q].type = (uint8_t)(seg[q] % T);
            out->run[q].zone = (uint8_t)(seg[q] / T);
            out->run[q].tp_idx = (uint8_t)k.tpi;
            out->run[q].n_stages = (uint8_t)(e - a);
        }
        return true;
    }
    return false;
}

}  // namespace sailor
