// Explicit batches of plan records (Sailor Sec. 4.3): the kernel behind sailor_simulate.
//
// A record costs 72 bytes in and 28 bytes out, so the batch is bound by HBM only if a record takes a few hundred
// instructions.  Three things keep it there:
//   - everything a stretch of equal stages needs (f + b, update time, gradient bytes, memory with and without an
//     in-flight microbatch) sits in ONE 32-byte table entry (one memory sector) per (stage make-up, GPU type, tp,
//     mbs, rc), the gradient bytes in a table per (stage make-up, tp), both formed once per context with the same functions and operation order as a stage-by-stage walk;
//   - the doubled one-way message time of every link (inside a node, between nodes, between zones) is tabulated
//     per microbatch size, so a stage boundary is one or two loads and at most one maximum;
//   - index arithmetic is 32 bits wide, and the GPUs a plan takes of a (zone, type) are added up over its runs only
//     when a run repeats an earlier run's (zone, type): no per-thread counters, so little shared memory and a large L1
//     for the table entries.
// The sums whose order of additions is part of the result (stage times, price rate, transfer cost) are still
// added one stage after the other, exactly as simulate_runs does, so both give the same bits.
#pragma once

#include "sailor_plan_kernels.cuh"

namespace sailor {

struct alignas(32) PieceRec {        // one per (composition, type, tp index, mbs index, rc): one 32-byte sector
    double fb;                       // f + b (+ f with recomputation) of a stage of this make-up
    double upd;                      // its update time
    uint64_t mem0r;                  // model + working bytes + the type's reserved bytes
    uint64_t mem1;                   // bytes kept per in-flight microbatch
};
static_assert(sizeof(PieceRec) == 32, "two 16-byte loads from one sector");

__host__ __device__ inline size_t piece_count(const TabHdr& h) {
    return (size_t)4 * h.chain_len * h.T * h.n_tp * h.n_mbs * 2;
}

// One thread per table entry; then the link tables (2 x one-way time per digit or zone pair and mbs index).
__global__ void batch_tables_kernel(unsigned char* blob) {
    TabView v;
    v.bind(blob, blob);
    const TabHdr* h = v.h;
    const size_t total = piece_count(*h);
    PieceRec* out = reinterpret_cast<PieceRec*>(blob + h->off_piece);
    for (size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x; x < total; x += (size_t)gridDim.x * blockDim.x) {
        size_t y = x;
        const uint32_t rc = y % 2; y /= 2;
        const uint32_t mi = y % h->n_mbs; y /= h->n_mbs;
        const uint32_t tpi = y % h->n_tp; y /= h->n_tp;
        const uint32_t g = y % h->T; y /= h->T;
        const size_t comp = y;
        const uint32_t nb = (uint32_t)(comp % h->chain_len), eh = (uint32_t)(comp / h->chain_len);
        const bool e = eh & 2u, hd = eh & 1u;
        const StageTimes st = stage_times(v, g, tpi, mi, nb, e, hd);
        const double b = rc ? add_rn(st.b, st.f) : st.b;
        const StageMem one = stage_memory(v, tpi, mi, rc, nb, e, hd, 1);     // model + 1 * kept + work
        const StageMem zero = stage_memory(v, tpi, mi, rc, nb, e, hd, 0);    // model + work
        PieceRec r;
        r.fb = add_rn(st.f, b);
        r.upd = st.u;
        r.mem0r = zero.mem + h->reserved[g];
        r.mem1 = one.mem - zero.mem;
        out[x] = r;
    }
    double* intra2 = reinterpret_cast<double*>(blob + h->off_lnk_intra2);
    double* inter2 = reinterpret_cast<double*>(blob + h->off_lnk_inter2);
    double* zone2 = reinterpret_cast<double*>(blob + h->off_lnk_zone2);
    const uint32_t n_d = h->R * h->n_mbs, n_z = h->Z * h->Z * h->n_mbs;
    for (uint32_t x = blockIdx.x * blockDim.x + threadIdx.x; x < 2 * n_d + n_z; x += gridDim.x * blockDim.x) {
        if (x < 2 * n_d) {
            const uint32_t y = x < n_d ? x : x - n_d, d = y / h->n_mbs, mi = y % h->n_mbs;
            const double msg = (double)v.p2p[mi];
            if (x < n_d) intra2[y] = mul_rn(2.0, link_time(v.intra_a[d], v.intra_i[d], v.intra_p, d, msg));
            else inter2[y] = mul_rn(2.0, link_time(v.inter_a[d], v.inter_i[d], v.inter_p, d, msg));
        } else {
            const uint32_t y = x - 2 * n_d, zz = y / h->n_mbs, mi = y % h->n_mbs;
            zone2[y] = mul_rn(2.0, link_time(v.zone_a[zz], v.zone_i[zz], v.zone_p, zz, (double)v.p2p[mi]));
        }
    }
}

// What the batch kernel keeps in shared memory of the context (a few hundred bytes, plain loads).
struct BatchConst {
    uint32_t T, Z, R, n_tp, n_mbs, chain_len, n_blocks, has_embed, has_head, heads_ok, has_poly;
    uint32_t piece_stride;           // entries per composition: T * n_tp * n_mbs * 2
    uint64_t gbs;
    uint32_t tp_values[SAILOR_TP_MAX];
    uint32_t mbs_values[SAILOR_MBS_MAX];
    uint32_t gpn[SAILOR_T_MAX];
    uint64_t cap[SAILOR_T_MAX];
    uint64_t p2p[SAILOR_MBS_MAX];
    uint32_t avail[R_MAX];
    double price_s[R_MAX];
    double egress[SAILOR_Z_MAX * SAILOR_Z_MAX];
    double intra_a[R_MAX], intra_i[R_MAX], inter_a[R_MAX], inter_i[R_MAX];
};

constexpr unsigned int SIM_ERR_DEVICE = 1u, SIM_ERR_BAD_RECORD = 2u;   // bits of the batch kernels' error word
constexpr int BATCH_THREADS = 256;
constexpr int BATCH_BLOCKS_PER_SM = 3;
constexpr uint32_t BATCH_POOL = 512;             // records a block stages and orders at a time
constexpr uint32_t REC_WORDS = sizeof(sailor_plan_rec) / 8;
static_assert(BATCH_POOL % BATCH_THREADS == 0, "every thread ranks BATCH_POOL / BATCH_THREADS records of a pool: a pool that is not a multiple leaves records unranked");

struct BatchOut {
    double t_iter, cost;
    uint64_t peak;
    uint32_t status;
};

// One record, held as nine 64-bit words at `w` (shared memory).  Follows simulate_runs operation by operation
// where roundings are concerned.
__device__ __forceinline__ BatchOut simulate_batch_record(const BatchConst& k, const TabView& v, const PieceRec* __restrict__ piece,
                                                          const double* __restrict__ intra2, const double* __restrict__ inter2,
                                                          const double* __restrict__ zone2, const uint64_t* w) {
    BatchOut o;
    o.t_iter = o.cost = make_nan();
    o.peak = 0;
    o.status = SAILOR_ST_BAD_RECORD;
    const uint64_t w0 = w[0];
    const uint32_t P = (uint32_t)w0 & 0xff, mi = (uint32_t)(w0 >> 8) & 0xff, rc = ((uint32_t)(w0 >> 16) & 0xff) ? 1u : 0u;
    const uint32_t n_runs = (uint32_t)(w0 >> 24) & 0xff, D = (uint32_t)(w0 >> 32) & 0xffff;
    if (P < 1 || P > SAILOR_P_MAX || n_runs < 1 || n_runs > SAILOR_RUN_MAX || D < 1 || mi >= k.n_mbs) return o;
    auto run_of_q = [&](uint32_t q) { return (uint32_t)(w[1 + (q >> 1)] >> (32 * (q & 1))); };

    // every index is checked before any table is read through it; GPUs taken per (zone, type) on the way
    uint32_t tot = 0, status = 0;
    bool bad = false;
    uint64_t seen = 0;
    for (uint32_t q = 0; q < n_runs; ++q) {
        const uint32_t r = run_of_q(q);
        const uint32_t g = r & 0xff, z = (r >> 8) & 0xff, tpi = (r >> 16) & 0xff, n = r >> 24;
        const bool ok = g < k.T && z < k.Z && tpi < k.n_tp && n >= 1;
        bad |= !ok;
        tot += n;
        if (ok) {
            const uint32_t tp = k.tp_values[tpi], d = z * k.T + g;
            if (tp > k.gpn[g] || !((k.heads_ok >> tpi) & 1u)) status |= SAILOR_ST_INVALID;
            uint64_t sum = (uint64_t)D * tp * n;            // GPUs this run takes of its (zone, type) ...
            if ((seen >> d) & 1ull)                          // ... and, rarely, what earlier runs took of the same
                for (uint32_t q2 = 0; q2 < q; ++q2) {
                    const uint32_t r2 = run_of_q(q2);
                    const uint32_t t2 = (r2 >> 16) & 0xff;
                    if ((r2 & 0xffff) == (r & 0xffff) && t2 < k.n_tp) sum += (uint64_t)D * k.tp_values[t2] * (r2 >> 24);
                }
            seen |= 1ull << d;
            if (sum > k.avail[d]) status |= SAILOR_ST_OVER_AVAIL;     // the total only grows from run to run
        }
    }
    if (bad || tot != P) return o;

    const uint32_t mbs = k.mbs_values[mi];
    const uint64_t dm = (uint64_t)D * mbs;
    uint64_t n_b;
    if (((k.gbs | dm) >> 32) == 0) {                        // the usual case: a 32-bit division
        const uint32_t q32 = (uint32_t)k.gbs / (uint32_t)dm;
        n_b = q32;
        if (q32 * (uint32_t)dm != (uint32_t)k.gbs) status |= SAILOR_ST_INVALID;
    } else {
        n_b = k.gbs / dm;
        if (n_b * dm != k.gbs) status |= SAILOR_ST_INVALID;
    }
    const uint32_t base = k.n_blocks / P, extra = k.n_blocks - base * P;
    const double xbytes = (double)(2 * n_b * (uint64_t)D * k.p2p[mi]);
    const double steps = (double)(2 * (uint64_t)(D - 1));
    const double coef = D > 1 ? steps / (double)D : 0.0;    // ring all-reduce: 2(D-1)/D
    double sum_t = 0.0, max_t = 0.0, max_sync = 0.0, max_u = 0.0, rate = 0.0, c_comm = 0.0;
    uint64_t peak = 0;
    bool oom = false;

    uint32_t i = 0;
    for (uint32_t q = 0; q < n_runs; ++q) {
        const uint32_t r = run_of_q(q);
        const uint32_t g = r & 0xff, z = (r >> 8) & 0xff, tpi = (r >> 16) & 0xff, run_end = i + (r >> 24);
        const uint32_t tp = k.tp_values[tpi], d = z * k.T + g;
        const double gpu_rate = mul_rn((double)(D * tp), k.price_s[d]);
        const bool intra_self = (uint64_t)D * (tp + tp) <= k.gpn[g];             // two neighbouring stages share a node
        const double c2_self = intra_self ? __ldg(&intra2[d * k.n_mbs + mi]) : __ldg(&inter2[d * k.n_mbs + mi]);
        const bool intra_dp = (uint64_t)D * tp <= k.gpn[g];
        const double ar_alpha = intra_dp ? k.intra_a[d] : k.inter_a[d], ar_inv = intra_dp ? k.intra_i[d] : k.inter_i[d];
        const uint32_t ent = ((g * k.n_tp + tpi) * k.n_mbs + mi) * 2 + rc;        // entry within a composition
        const uint64_t cap = k.cap[g];
        while (i < run_end) {
            const bool e = (i == 0) && k.has_embed, hd = (i == P - 1) && k.has_head;
            // the piece ends with the run, after the embedding stage, where the extra blocks run out, before the head stage
            uint32_t piece_end = run_end;
            if (e) piece_end = 1;
            else {
                if (i < extra && extra < piece_end) piece_end = extra;
                if (k.has_head && i < P - 1 && P - 1 < piece_end) piece_end = P - 1;
            }
            const uint32_t comp = ((e ? 2u : 0u) + (hd ? 1u : 0u)) * k.chain_len + base + (i < extra ? 1u : 0u);
            const PieceRec* pr = piece + (size_t)comp * k.piece_stride + ent;
            const double2 a0 = __ldg(reinterpret_cast<const double2*>(pr));                // fb, upd
            const ulonglong2 a1 = __ldg(reinterpret_cast<const ulonglong2*>(pr) + 1);      // mem0r, mem1
            const double fb = a0.x;
            if (D > 1) {
                const double grad = __ldg(&v.cmp_grad[comp * k.n_tp + tpi]);
                const double volume = mul_rn(coef, grad);
                double t;
                if (k.has_poly) {
                    const double* poly = intra_dp ? v.intra_p : v.inter_p;
                    t = poly ? volume / poly_bw(poly + 4 * d, grad / (double)D) : mul_rn(volume, ar_inv);
                } else t = mul_rn(volume, ar_inv);
                max_sync = dmax(max_sync, add_rn(t, mul_rn(steps, ar_alpha)));
            }
            const uint64_t left = P - i, inflight = left < n_b ? left : n_b;
            const uint64_t m = a1.x + inflight * a1.y;
            oom |= m > cap;
            peak = m > peak ? m : peak;
            max_u = dmax(max_u, a0.y);
            const bool closes = piece_end == run_end;          // the piece's last stage sends to the next run, or is the final stage
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
                double t = fb;                                  // the final stage sends nothing: fb + 2*0
                if (piece_end < P) {                            // the next stage opens run q + 1
                    const uint32_t nx = run_of_q(q + 1);
                    const uint32_t g2 = nx & 0xff, z2 = (nx >> 8) & 0xff, tp2 = k.tp_values[(nx >> 16) & 0xff];
                    double c2;
                    if (z2 != z) {
                        c2 = __ldg(&zone2[(z * k.Z + z2) * k.n_mbs + mi]);
                        c_comm = add_rn(c_comm, mul_rn(xbytes, k.egress[z * k.Z + z2]));
                    } else if (g2 == g && (uint64_t)D * (tp + tp2) <= k.gpn[g]) {
                        c2 = __ldg(&intra2[d * k.n_mbs + mi]);
                    } else {
                        c2 = dmax(__ldg(&inter2[d * k.n_mbs + mi]), __ldg(&inter2[(z * k.T + g2) * k.n_mbs + mi]));
                    }
                    t = add_rn(fb, c2);
                }
                sum_t = add_rn(sum_t, t);
                max_t = dmax(max_t, t);
                rate = add_rn(rate, gpu_rate);
            }
            i = piece_end;
        }
    }
    if (oom) status |= SAILOR_ST_OOM;
    o.peak = peak;
    o.status = status;
    if (status & SAILOR_ST_INVALID) return o;
    const double t_pp = add_rn(sum_t, mul_rn((double)n_b, max_t));
    o.t_iter = add_rn(add_rn(t_pp, max_sync), max_u);
    o.cost = add_rn(mul_rn(rate, o.t_iter), c_comm);
    return o;
}

// A block stages a pool of records in shared memory with coalesced 8-byte loads, orders it by run count and
// stage count (the work of a record grows with both; any order gives the same results), and its warps take groups
// of 32 similar records from the pool, longest first, until it is empty.  Results leave as four
// structure-of-arrays streams.
__global__ void __launch_bounds__(BATCH_THREADS, BATCH_BLOCKS_PER_SM)
simulate_kernel(const unsigned char* __restrict__ blob, const uint16_t* __restrict__ avail,
                const sailor_plan_rec* __restrict__ plans, uint64_t n, double* __restrict__ t_iter,
                uint64_t* __restrict__ peak_mem, double* __restrict__ cost, uint32_t* __restrict__ status,
                unsigned int* bad_flag) {                      // not null: set SIM_ERR_BAD_RECORD there when a record is refused
    __shared__ BatchConst k;
    __shared__ uint64_t recs[BATCH_POOL * REC_WORDS];
    __shared__ uint32_t hist[256];
    __shared__ uint16_t perm[BATCH_POOL];
    __shared__ uint32_t next_group;
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    TabView v;
    v.bind(blob, blob);                                        // everything read through it comes from global memory
    const TabHdr* h = v.h;
    if (tid == 0) {
        k.T = h->T; k.Z = h->Z; k.R = h->R; k.n_tp = h->n_tp; k.n_mbs = h->n_mbs; k.chain_len = h->chain_len;
        k.n_blocks = h->n_blocks; k.has_embed = h->has_embed; k.has_head = h->has_head; k.heads_ok = h->heads_ok;
        k.has_poly = (h->off_intra_p | h->off_inter_p) ? 1u : 0u;
        k.piece_stride = h->T * h->n_tp * h->n_mbs * 2;
        k.gbs = h->gbs;
    }
    if (tid < SAILOR_TP_MAX) k.tp_values[tid] = h->tp_values[tid];
    if (tid < SAILOR_MBS_MAX) { k.mbs_values[tid] = h->mbs_values[tid]; k.p2p[tid] = tid < h->n_mbs ? v.p2p[tid] : 0; }
    if (tid < SAILOR_T_MAX) { k.gpn[tid] = h->gpn[tid]; k.cap[tid] = h->capacity[tid]; }
    if (tid < h->R) {
        k.avail[tid] = avail[tid];
        k.price_s[tid] = v.price_s[tid];
        k.intra_a[tid] = v.intra_a[tid]; k.intra_i[tid] = v.intra_i[tid];
        k.inter_a[tid] = v.inter_a[tid]; k.inter_i[tid] = v.inter_i[tid];
    }
    if (tid < h->Z * h->Z) k.egress[tid] = v.egress[tid];
    const PieceRec* piece = reinterpret_cast<const PieceRec*>(blob + h->off_piece);
    const double* intra2 = reinterpret_cast<const double*>(blob + h->off_lnk_intra2);
    const double* inter2 = reinterpret_cast<const double*>(blob + h->off_lnk_inter2);
    const double* zone2 = reinterpret_cast<const double*>(blob + h->off_lnk_zone2);
    const uint64_t* src = reinterpret_cast<const uint64_t*>(plans);
    for (uint64_t pool = (uint64_t)blockIdx.x * BATCH_POOL; pool < n; pool += (uint64_t)gridDim.x * BATCH_POOL) {
        const uint32_t cnt = (uint32_t)(n - pool < BATCH_POOL ? n - pool : BATCH_POOL);
        __syncthreads();
        for (uint32_t x = tid; x < cnt * REC_WORDS; x += BATCH_THREADS) recs[x] = __ldcs(&src[pool * REC_WORDS + x]);
        hist[tid] = 0;
        if (tid == 0) next_group = 0;
        __syncthreads();
        // counting sort, most work first: by run count (byte 3 of a record), then by stage count (byte 0)
        uint32_t key[BATCH_POOL / BATCH_THREADS], rank[BATCH_POOL / BATCH_THREADS];
#pragma unroll
        for (uint32_t u = 0; u < BATCH_POOL / BATCH_THREADS; ++u) {
            const uint32_t x = tid + u * BATCH_THREADS;
            key[u] = rank[u] = 0;
            if (x < cnt) {
                const uint32_t w0 = (uint32_t)recs[x * REC_WORDS];
                const uint32_t P = w0 & 0xff, nr = w0 >> 24;
                const uint32_t work = (nr > 15u ? 15u : nr) * 16u + (P > 95u ? 15u : P / 6u);
                key[u] = 255u - work;
                rank[u] = atomicAdd(&hist[key[u]], 1u);
            }
        }
        __syncthreads();
        if (tid < 32) {                                        // exclusive scan of the 256 bins by one warp
            uint32_t h4[8], sum = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) { h4[q] = hist[tid * 8 + q]; sum += h4[q]; }
            uint32_t incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t up = __shfl_up_sync(FULL, incl, o);
                if (tid >= (uint32_t)o) incl += up;
            }
            uint32_t at = incl - sum;
#pragma unroll
            for (int q = 0; q < 8; ++q) { hist[tid * 8 + q] = at; at += h4[q]; }
        }
        __syncthreads();
#pragma unroll
        for (uint32_t u = 0; u < BATCH_POOL / BATCH_THREADS; ++u) {
            const uint32_t x = tid + u * BATCH_THREADS;
            if (x < cnt) perm[hist[key[u]] + rank[u]] = (uint16_t)x;
        }
        __syncthreads();
        const uint32_t n_groups = (cnt + 31) / 32;
        for (;;) {                                             // warps drain the pool, longest records first
            uint32_t grp = 0;
            if (lane == 0) grp = atomicAdd(&next_group, 1u);
            grp = __shfl_sync(FULL, grp, 0);
            if (grp >= n_groups) break;
            const uint32_t slot = grp * 32 + lane;
            if (slot < cnt) {
                const uint32_t mine = perm[slot];
                const BatchOut o = simulate_batch_record(k, v, piece, intra2, inter2, zone2, &recs[mine * REC_WORDS]);
                if (t_iter) __stcs(&t_iter[pool + mine], o.t_iter);
                if (peak_mem) __stcs(&peak_mem[pool + mine], o.peak);
                if (cost) __stcs(&cost[pool + mine], o.cost);
                if (status) __stcs(&status[pool + mine], o.status);
                if (bad_flag && (o.status & SAILOR_ST_BAD_RECORD)) atomicOr(bad_flag, SIM_ERR_BAD_RECORD);
            }
            __syncwarp();
        }
    }
}

}  // namespace sailor
