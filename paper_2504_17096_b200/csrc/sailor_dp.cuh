// Per-stage GPU types by dynamic programming (Sailor Sec. 4.2.2: Eq. 1 and T_total).
//
// A problem is one configuration (P, mbs, tp, rc, D) with one zone order.  Its states are
// (stage i, type g of stage i, zone position zp of stage i, u = stages per type already placed in
// that zone, stage i included).  Zones before zp are never revisited and zones after it are
// untouched (first fit), so nothing else of the past matters.  A type that a zone could give to all
// P stages is not counted in u.  For every zone position and type there is a slice of S[zp] entries
// indexed by u, in one of two ways chosen per zone position: densely in mixed radix (radix cap + 1 per
// counted type), or compactly by the rank of u among the count vectors that respect the caps and add
// up to at most P (a zone never holds more than P stages); the compact index is much smaller when
// many types are scarce at once.  The value of a state is the best plan of stages i.. from it:
// (sum of stage times, straggler, slowest synchronisation, slowest update).
//
// The tables are filled from the last stage to the first.  One launch handles one stage distance
// from the end for every problem of a batch (problems are sorted by depth, so the launch for
// distance s covers a prefix of the block list); a thread owns one state and tries every type for
// the next stage.  Per-configuration quantities (stage times per type, synchronisation per digit,
// message times per digit pair) are formed once per configuration by dp_tables_kernel.
#pragma once

#include "sailor_plan_kernels.cuh"

namespace sailor {

constexpr int DP_THREADS = 256;
constexpr uint8_t DP_NONE = 255;
constexpr uint32_t DP_DENSE = 0xffffffffu;

struct alignas(32) DpVal {           // best plan of stages i.. from a state; sum = +inf: there is none.  Aligned to its
                                     // size: a value then moves in one load or store
    double sum, mx, sy, up;
};

struct DpProblem {
    uint64_t val_off;                // first entry of this problem in the two level buffers of its batch
    uint64_t choice_off;             // first byte of its choices: [stage][entry]
    uint32_t config, order, index;   // index = config * n_orders + order
    uint32_t n_lvl;                  // entries per stage
    uint32_t P, nz, need;            // need = D * tp GPUs per stage
    uint8_t zone[SAILOR_Z_MAX];      // zone of each position of the order
    uint8_t cap[SAILOR_Z_MAX][SAILOR_T_MAX];       // stages a (position, type) can host, saturated at 255
    uint8_t first_later[SAILOR_Z_MAX][SAILOR_T_MAX];   // first position after zp that can host a stage of the type
    uint32_t stride[SAILOR_Z_MAX][SAILOR_T_MAX];   // mixed-radix stride of a counted type; 0: not counted
    uint32_t S[SAILOR_Z_MAX];        // entries of one (position, type) slice
    uint32_t zp_base[SAILOR_Z_MAX + 1];            // first entry of each position's T slices
    uint32_t vt_lo;                  // the problem's rank tables are vtabs[vt_lo .. vt_lo + vt_len)
    uint32_t first_idx[SAILOR_Z_MAX][SAILOR_T_MAX];    // index of "one stage, of this type" inside a slice
    uint32_t vt_off[SAILOR_Z_MAX];   // compact index: offset of the position's rank table in `vtabs`; DP_DENSE: mixed radix
    uint32_t rank_off[SAILOR_Z_MAX]; // the position's rank table whatever its index (DP_DENSE: no counted type, or
                                     // none built): lets a launch enumerate only the count vectors a stage can reach
    uint32_t vt_len, _pad;
    uint8_t n_counted[SAILOR_Z_MAX]; // counted types of each position
    uint64_t magic[SAILOR_Z_MAX][SAILOR_T_MAX];    // ceil(2^64 / (cap + 1)) of a counted type: for 32-bit x,
                                                   // x / (cap + 1) == high 64 bits of x * magic
};
static_assert(sizeof(DpProblem) % 8 == 0, "copied word by word");

struct DpResult {                    // per problem, written by dp_finish_kernel
    double value;                    // +inf: no plan
    double t_iter, cost;             // the simulator's figures for the plan (stage order)
    uint64_t peak_mem;
    uint32_t status, _pad;
    uint8_t type[SAILOR_P_MAX];
    uint8_t zone[SAILOR_P_MAX];
};

// Per-configuration tables in global memory, one block of `stride` doubles per configuration:
//   fb[p_max][T], upd[p_max][T], sync[p_max][R], c2x[R][R] (2 * message time, [next digit][this digit]),
//   then ok[p_max] (u32 bit g: stage fits type g and tp fits its node), n_b (u64), valid (u32).
struct DpTabLayout {
    uint32_t p_max, T, R;
    __host__ __device__ size_t off_fb() const { return 0; }
    __host__ __device__ size_t off_upd() const { return (size_t)p_max * T; }
    __host__ __device__ size_t off_sync() const { return 2 * (size_t)p_max * T; }
    __host__ __device__ size_t off_c2x() const { return 2 * (size_t)p_max * T + (size_t)p_max * R; }
    __host__ __device__ size_t off_ok() const { return off_c2x() + (size_t)R * R; }               // in doubles
    __host__ __device__ size_t off_nb() const { return off_ok() + (p_max + 1) / 2; }
    __host__ __device__ size_t stride() const { return off_nb() + 2; }
};

__global__ void __launch_bounds__(DP_THREADS)
dp_tables_kernel(const unsigned char* __restrict__ blob, SpaceDesc sp, uint32_t n_config, DpTabLayout lay,
                 double* __restrict__ tabs) {
    __shared__ uint64_t s_params[SAILOR_P_MAX];
    __shared__ uint32_t s_ok[SAILOR_P_MAX];
    TabView v;
    v.bind(blob, blob);
    const TabHdr* h = v.h;
    const uint32_t T = h->T, R = h->R, tid = threadIdx.x;
    for (uint32_t c = blockIdx.x; c < n_config; c += gridDim.x) {
        __syncthreads();
        const Config k = config_of(sp, c);
        double* tab = tabs + (size_t)c * lay.stride();
        const uint32_t tp = h->tp_values[k.tpi];
        const uint64_t dm = (uint64_t)k.D * h->mbs_values[k.mi];
        const bool valid = k.D >= 1 && h->gbs % dm == 0 && h->heads % tp == 0;
        const uint64_t n_b = valid ? h->gbs / dm : 0;
        if (tid == 0) {
            *reinterpret_cast<uint64_t*>(tab + lay.off_nb()) = n_b;
            *reinterpret_cast<uint32_t*>(tab + lay.off_nb() + 1) = valid ? 1u : 0u;
        }
        for (uint32_t i = tid; i < SAILOR_P_MAX; i += DP_THREADS) s_ok[i] = 0;
        __syncthreads();
        if (!valid) continue;
        const uint32_t P = k.P, base = h->n_blocks / P, extra = h->n_blocks % P;
        for (uint32_t x = tid; x < P * T; x += DP_THREADS) {
            const uint32_t i = x / T, g = x % T;
            const uint32_t nb = base + (i < extra ? 1u : 0u);
            const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
            const StageTimes st = stage_times(v, g, k.tpi, k.mi, nb, e, hd);
            const double b = k.rc ? add_rn(st.b, st.f) : st.b;
            tab[lay.off_fb() + x] = add_rn(st.f, b);
            tab[lay.off_upd() + x] = st.u;
            const uint64_t inflight = (uint64_t)(P - i) < n_b ? (uint64_t)(P - i) : n_b;
            const StageMem sm = stage_memory(v, k.tpi, k.mi, k.rc, nb, e, hd, inflight);
            if (sm.mem + h->reserved[g] <= h->capacity[g] && tp <= h->gpn[g]) atomicOr(&s_ok[i], 1u << g);
            if (g == 0) s_params[i] = sm.params;
        }
        __syncthreads();
        const double steps = (double)(2 * (uint64_t)(k.D - 1)), coef = steps / (double)k.D;
        for (uint32_t x = tid; x < P * R; x += DP_THREADS) {
            const uint32_t i = x / R, d = x % R;
            tab[lay.off_sync() + x] = k.D > 1 ? allreduce_time(v, d % T, d, tp, k.D, s_params[i], steps, coef) : 0.0;
        }
        const double msg = (double)v.p2p[k.mi];
        for (uint32_t x = tid; x < R * R; x += DP_THREADS) {
            const uint32_t dn = x / R, d = x % R;          // [next][this]
            tab[lay.off_c2x() + x] = mul_rn(2.0, boundary_time(v, d % T, d / T, tp, dn % T, dn / T, tp, k.D, msg));
        }
        for (uint32_t i = tid; i < P; i += DP_THREADS) reinterpret_cast<uint32_t*>(tab + lay.off_ok())[i] = s_ok[i];
    }
}

// ---- the index of a count vector inside a slice -------------------------------------------------------
//
// Compact index of zone position zp: the counted types j = 0 .. m-1 (ascending type) have caps c_j.  With
// W[j][s] = number of (u_j .. u_{m-1}) within the caps that add up to at most s, and V[j][s] = W[j][0] + .. +
// W[j][s], the rank of u in lexicographic order is sum_j (V[j+1][s_j] - V[j+1][s_j - u_j]), s_0 = P,
// s_{j+1} = s_j - u_j.  The table holds V[j][s] for j = 0 .. m, s = 0 .. P, row after row.

// One digit of an unranking: the count x of a type, given the rank r among the vectors that agree on the types
// before it and have s stages left for this type and the later ones.  `row` = V[j + 1][.] of the type's successor:
// below(x) = row[s] - row[s - x] vectors start with a smaller count, and x is the largest count <= lim with
// below(x) <= r.  After the last counted type nothing varies (V = s + 1), so below(x) = x there; elsewhere below is
// non-decreasing in x and a bisection finds x.
__device__ __forceinline__ void dp_digit(const uint32_t* __restrict__ row, uint32_t s, uint32_t lim, uint32_t r, bool last,
                                         uint32_t& x, uint32_t& below) {
    if (last) {
        x = min(lim, r);
        below = x;
        return;
    }
    const uint32_t top = row[s];
    uint32_t lo = 0, hi = lim;
    while (lo < hi) {
        const uint32_t mid = (lo + hi + 1) >> 1;                 // 1 <= mid <= lim <= s
        if (top - row[s - mid] <= r) lo = mid; else hi = mid - 1;
    }
    x = lo;
    below = lo ? top - row[s - lo] : 0u;
}

// counts of a slice index: u[t] for counted types, 0 for the others.  Returns false, possibly before all counts
// are known, as soon as they add up to more than `limit`.
__device__ __forceinline__ bool dp_counts(const DpProblem& pb, const uint32_t* __restrict__ vtabs, uint32_t zp, uint32_t T,
                                          uint32_t ui, uint32_t (&u)[SAILOR_T_MAX], uint32_t limit) {
    uint32_t total = 0;
    if (pb.vt_off[zp] == DP_DENSE) {
        uint32_t rem = ui;
#pragma unroll
        for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) {
            u[t] = 0;
            if (t < T && pb.stride[zp][t]) {
                const uint32_t q = (uint32_t)__umul64hi((uint64_t)rem, pb.magic[zp][t]);
                u[t] = rem - q * (pb.cap[zp][t] + 1u);
                rem = q;
                total += u[t];
            }
        }
        return total <= limit;
    } else {
        const uint32_t* vt = vtabs + pb.vt_off[zp];
        const uint32_t w = pb.P + 1;
        uint32_t r = ui, s = pb.P, j = 0;
#pragma unroll
        for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) {
            u[t] = 0;
            if (t < T && pb.stride[zp][t]) {
                const uint32_t lim = min((uint32_t)pb.cap[zp][t], s);
                uint32_t x, below;                               // `below`: vectors that start with a count smaller than x
                dp_digit(vt + (j + 1) * w, s, lim, r, j + 1 == pb.n_counted[zp], x, below);
                u[t] = x;
                total += x;
                if (total > limit) return false;                 // the walks of the remaining types are not needed
                r -= below;
                s -= x;
                ++j;
            }
        }
        return true;
    }
}

// The r-th count vector (lexicographic) among those within the caps that add up to at most `budget`.
__device__ __forceinline__ void dp_unrank(const DpProblem& pb, const uint32_t* __restrict__ vt, uint32_t zp, uint32_t T,
                                          uint32_t r, uint32_t budget, uint32_t (&u)[SAILOR_T_MAX]) {
    const uint32_t w = pb.P + 1;
    uint32_t s = budget, j = 0;
#pragma unroll
    for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) {
        u[t] = 0;
        if (t < T && pb.stride[zp][t]) {
            const uint32_t lim = min((uint32_t)pb.cap[zp][t], s);
            uint32_t x, below;
            dp_digit(vt + (j + 1) * w, s, lim, r, j + 1 == pb.n_counted[zp], x, below);
            u[t] = x;
            r -= below;
            s -= x;
            ++j;
        }
    }
}

// slice index of the count vector u with one more stage of type `plus_one` (compact index only)
__device__ __forceinline__ uint32_t dp_rank(const DpProblem& pb, const uint32_t* __restrict__ vtabs, uint32_t zp, uint32_t T,
                                            const uint32_t (&u)[SAILOR_T_MAX], uint32_t plus_one) {
    const uint32_t* vt = vtabs + pb.vt_off[zp];
    const uint32_t w = pb.P + 1;
    uint32_t r = 0, s = pb.P, j = 0;
#pragma unroll
    for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) {
        if (t < T && pb.stride[zp][t]) {
            const uint32_t x = u[t] + (t == plus_one ? 1u : 0u);
            const uint32_t* row = vt + (j + 1) * w;
            if (x) r += row[s] - row[s - x];                     // the caller keeps the counts within P in total
            s -= x;
            ++j;
        }
    }
    return r;
}

// Where does a stage of type g2 go when the previous stage sits at position zp with counts u (slice index ui)?
// Returns the position (DP_NONE: nowhere) and the entry index of the state that results.
struct DpMove { uint32_t zp, entry; };

__device__ __forceinline__ DpMove dp_move(const DpProblem& pb, const uint32_t* __restrict__ vtabs, uint32_t T, uint32_t zp,
                                          uint32_t ui, const uint32_t (&u)[SAILOR_T_MAX], uint32_t g2) {
    DpMove m;
    const uint32_t cap = pb.cap[zp][g2];
    uint32_t u_g2 = 0, placed = 0;
#pragma unroll
    for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) {
        u_g2 = t == g2 ? u[t] : u_g2;
        placed += u[t];
    }
    // first fit: this zone while it has room for one more stage of the type, else the next zone that has
    const bool counted = pb.stride[zp][g2] != 0;
    const bool here = counted ? u_g2 < cap : cap >= 1;           // not counted: room for every stage, or none at all
    if (here) {
        m.zp = zp;
        uint32_t idx = ui;
        if (counted) {
            if (pb.vt_off[zp] == DP_DENSE) idx = ui + pb.stride[zp][g2];
            else if (placed >= pb.P) { m.zp = DP_NONE; m.entry = 0; return m; }      // more than P stages: no such state
            else idx = dp_rank(pb, vtabs, zp, T, u, g2);
        }
        m.entry = pb.zp_base[zp] + g2 * pb.S[zp] + idx;
        return m;
    }
    const uint32_t p = pb.first_later[zp][g2];
    m.zp = p;
    m.entry = p == DP_NONE ? 0u : pb.zp_base[p] + g2 * pb.S[p] + pb.first_idx[p][g2];      // the new zone holds this stage only
    return m;
}

struct DpLevelParams {
    const DpProblem* problems;
    const uint32_t* blk_problem;     // entries mode: block -> problem of the batch
    const uint32_t* blk_first;       // entries mode: block -> first entry it covers
    const uint32_t* blk_prefix;      // live mode: [n_active + 1] blocks before each problem of this launch
    uint32_t n_active;               // live mode: problems of this launch (a prefix of the batch)
    uint32_t per_thread;             // vector kernel: count vectors a thread takes, a block's width apart
    const double* tabs;
    const uint32_t* vtabs;           // rank tables of the compactly indexed zone positions
    DpVal* val[2];                   // level buffers; stage i lives in val[(P - 1 - i) & 1]
    uint8_t* choice;
    DpTabLayout lay;
    uint32_t T;
    uint32_t dist;                   // stage i = P - 1 - dist
};

// LIVE = false: a thread per table entry (block map over entries); entries no stage sequence can reach at this
// stage leave early.  LIVE = true: a thread per count vector that stage i can have reached (at most i + 1 stages
// in the zone), enumerated by rank with that budget through the positions' rank tables (block map over those).
template <bool LIVE>
__global__ void __launch_bounds__(DP_THREADS, 5) dp_level_kernel(const __grid_constant__ DpLevelParams lp) {
    __shared__ DpProblem pb;
    const uint32_t tid = threadIdx.x;
    uint32_t which, first;
    if (LIVE) {                                              // the problem whose blocks include this one (all threads alike)
        uint32_t lo = 0, hi = lp.n_active;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (lp.blk_prefix[mid] <= blockIdx.x) lo = mid; else hi = mid;
        }
        which = lo;
        first = (blockIdx.x - lp.blk_prefix[lo]) * DP_THREADS;
    } else {
        which = lp.blk_problem[blockIdx.x];
        first = lp.blk_first[blockIdx.x];
    }
    {
        const DpProblem* src = lp.problems + which;
        for (uint32_t x = tid; x < sizeof(DpProblem) / 4; x += DP_THREADS)
            reinterpret_cast<uint32_t*>(&pb)[x] = reinterpret_cast<const uint32_t*>(src)[x];
    }
    __syncthreads();
    const uint32_t T = lp.T, P = pb.P, i = P - 1 - lp.dist;
    const double* tab = lp.tabs + (size_t)pb.config * lp.lay.stride();
    const uint32_t* okv = reinterpret_cast<const uint32_t*>(tab + lp.lay.off_ok());
    const double nb = (double)*reinterpret_cast<const uint64_t*>(tab + lp.lay.off_nb());
    uint32_t zp = 0, g = 0, ui, e;
    uint32_t u[SAILOR_T_MAX];
    uint32_t S;
    if (LIVE) {
        // live index -> (zone position, type, r-th count vector with at most i + 1 stages) -> its table entry
        uint32_t l = first + tid;
        const uint32_t budget = i + 1;                       // <= P
        uint32_t wz = 0;
        for (;; ++zp) {
            if (zp == pb.nz) return;                             // past the last live vector of this stage
            wz = 1;
            if (pb.rank_off[zp] != DP_DENSE) {
                const uint32_t* row0 = lp.vtabs + pb.rank_off[zp];   // V[0][s]: vectors of all counted types up to sum s
                wz = row0[budget] - row0[budget - 1];
            }
            if (l < T * wz) break;
            l -= T * wz;
        }
        while (l >= wz) { l -= wz; ++g; }
        S = pb.S[zp];
        if (pb.rank_off[zp] != DP_DENSE) dp_unrank(pb, lp.vtabs + pb.rank_off[zp], zp, T, l, budget, u);
        else {
#pragma unroll
            for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) u[t] = 0;
        }
        if (pb.vt_off[zp] != DP_DENSE) ui = dp_rank(pb, lp.vtabs, zp, T, u, 0xffffffffu);
        else {
            ui = 0;
#pragma unroll
            for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) ui += (t < T) ? u[t] * pb.stride[zp][t] : 0u;
        }
        e = pb.zp_base[zp] + g * S + ui;
    } else {
        e = first + tid;
        if (e >= pb.n_lvl) return;
        // entry -> (zone position, type, counts); no division by run-time values: the slices of a position are
        // stepped through, and the counts come off by reciprocal multiplication or by a walk through the rank table
        while (zp + 1 < pb.nz && e >= pb.zp_base[zp + 1]) ++zp;
        ui = e - pb.zp_base[zp];
        S = pb.S[zp];
        while (ui >= S) { ui -= S; ++g; }
        // stage i is at most the (i+1)-th stage of its zone: entries that count more are never reached, and
        // since a move raises the count by one per stage, no entry that passes this test ever reads one that fails it
        if (!dp_counts(pb, lp.vtabs, zp, T, ui, u, i + 1)) return;
    }
    DpVal* cur = lp.val[lp.dist & 1] + pb.val_off;
    const DpVal* nxt = lp.val[(lp.dist & 1) ^ 1] + pb.val_off;
    uint8_t* choice = lp.choice + pb.choice_off + (size_t)i * pb.n_lvl;
    DpVal best;
    best.sum = make_inf(); best.mx = best.sy = best.up = 0.0;
    uint8_t pick = DP_NONE;
    // a state holds stage i itself: its type must be usable there and, when counted, counted at least once
    uint32_t u_g = 0;
#pragma unroll
    for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) u_g = t == g ? u[t] : u_g;
    const bool self = ((okv[i] >> g) & 1u) && pb.cap[zp][g] >= 1 && (pb.stride[zp][g] == 0 || u_g >= 1);
    if (self) {
        const uint32_t d = pb.zone[zp] * T + g;
        const double fb = tab[lp.lay.off_fb() + i * T + g], upd = tab[lp.lay.off_upd() + i * T + g];
        const double sync = tab[lp.lay.off_sync() + (size_t)i * lp.lay.R + d];
        if (lp.dist == 0) {                                      // the last stage sends nothing
            best.sum = fb; best.mx = fb; best.sy = sync; best.up = upd;
        } else {
            double best_v = make_inf();
            const uint32_t ok_next = okv[i + 1];
#pragma unroll
            for (uint32_t g2 = 0; g2 < SAILOR_T_MAX; ++g2) {
                if (g2 >= T) break;
                if (!((ok_next >> g2) & 1u)) continue;
                const DpMove mv = dp_move(pb, lp.vtabs, T, zp, ui, u, g2);
                if (mv.zp == DP_NONE) continue;
                const uint32_t zp2 = mv.zp, entry = mv.entry;
                const DpVal n = nxt[entry];
                if (!(n.sum < make_inf())) continue;
                const uint32_t d2 = pb.zone[zp2] * T + g2;
                const double t = add_rn(fb, tab[lp.lay.off_c2x() + (size_t)d2 * lp.lay.R + d]);
                DpVal c;
                c.sum = add_rn(t, n.sum);
                c.mx = dmax(t, n.mx);
                c.sy = dmax(sync, n.sy);
                c.up = dmax(upd, n.up);
                const double val = add_rn(add_rn(add_rn(c.sum, mul_rn(nb, c.mx)), c.sy), c.up);
                if (pick == DP_NONE || val < best_v) { best = c; best_v = val; pick = (uint8_t)g2; }
            }
        }
    }
    cur[e] = best;
    choice[e] = pick;
}

// A thread per reachable count vector, all types of stage i at once (TM >= T types).  The T entries that share a
// count vector share its unranking, its table index and, for every type of the next stage, the moved vector's entry:
// those are formed once, the next stage's values are gathered together, and only the T x T combinations remain per
// type.  Same arithmetic per (type, next type) pair and the same order of the next types as dp_level_kernel.

constexpr uint32_t DP_VEC_PER_THREAD = 4;       // in launches large enough to fill the GPU several times over

// The work of one stage (distance `dist` from the last) of the problem `pb` for the count vectors first + tid,
// first + DP_THREADS + tid, ... (`rounds` of them): see dp_level_vec_kernel.  `vtabs` addresses the problem's rank
// tables by their offsets from the start of all tables.
template <uint32_t TM>
__device__ __forceinline__ void dp_vec_level(const DpLevelParams& lp, const DpProblem& pb, const uint32_t* vtabs, uint32_t dist,
                                             uint32_t first, uint32_t rounds) {
    const uint32_t tid = threadIdx.x;
    const uint32_t T = lp.T, P = pb.P, i = P - 1 - dist;
    const double* tab = lp.tabs + (size_t)pb.config * lp.lay.stride();
    const uint32_t* okv = reinterpret_cast<const uint32_t*>(tab + lp.lay.off_ok());
    const double nb = (double)*reinterpret_cast<const uint64_t*>(tab + lp.lay.off_nb());
    DpVal* cur = lp.val[dist & 1] + pb.val_off;
    const DpVal* nxt = lp.val[(dist & 1) ^ 1] + pb.val_off;
    uint8_t* choice = lp.choice + pb.choice_off + (size_t)i * pb.n_lvl;
    const uint32_t budget = i + 1;                           // <= P
    const uint32_t ok_here = okv[i];
    // several vectors per thread, a block's width apart: the block's set-up (its problem, the rank tables) is paid once
    for (uint32_t round = 0; round < rounds; ++round) {
        uint32_t zp = 0, ui;
        uint32_t u[SAILOR_T_MAX];
        uint32_t l = first + round * DP_THREADS + tid;
        for (;; ++zp) {
            if (zp == pb.nz) return;                             // past the last reachable vector (later rounds too)
            uint32_t wz = 1;
            if (pb.rank_off[zp] != DP_DENSE) {
                const uint32_t* row0 = vtabs + pb.rank_off[zp];
                wz = row0[budget] - row0[budget - 1];
            }
            if (l < wz) break;
            l -= wz;
        }
        const uint32_t S = pb.S[zp];
        if (pb.rank_off[zp] != DP_DENSE) dp_unrank(pb, vtabs + pb.rank_off[zp], zp, T, l, budget, u);
        else {
#pragma unroll
            for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) u[t] = 0;
        }
        if (pb.vt_off[zp] != DP_DENSE) ui = dp_rank(pb, vtabs, zp, T, u, 0xffffffffu);
        else {
            ui = 0;
#pragma unroll
            for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) ui += (t < T) ? u[t] * pb.stride[zp][t] : 0u;
        }
        const uint32_t e0 = pb.zp_base[zp] + ui;
        // what follows a stage of each type g2: the entry it leads to (the same for every type of stage i) and its value
        DpVal n[TM];
        uint32_t d2v[TM];
#pragma unroll
        for (uint32_t g2 = 0; g2 < TM; ++g2) {
            d2v[g2] = DP_NONE;
            n[g2].sum = make_inf(); n[g2].mx = n[g2].sy = n[g2].up = 0.0;
        }
        if (dist != 0) {
            const uint32_t ok_next = okv[i + 1];
#pragma unroll
            for (uint32_t g2 = 0; g2 < TM; ++g2) {
                if (g2 >= T || !((ok_next >> g2) & 1u)) continue;
                const DpMove mv = dp_move(pb, vtabs, T, zp, ui, u, g2);
                if (mv.zp == DP_NONE) continue;
                n[g2] = nxt[mv.entry];
                d2v[g2] = pb.zone[mv.zp] * T + g2;
            }
        }
#pragma unroll
        for (uint32_t g = 0; g < TM; ++g) {
            if (g >= T) break;
            DpVal best;
            best.sum = make_inf(); best.mx = best.sy = best.up = 0.0;
            uint8_t pick = DP_NONE;
            // a state holds stage i itself: its type must be usable there and, when counted, counted at least once
            const bool self = ((ok_here >> g) & 1u) && pb.cap[zp][g] >= 1 && (pb.stride[zp][g] == 0 || u[g] >= 1);
            if (self) {
                const uint32_t d = pb.zone[zp] * T + g;
                const double fb = tab[lp.lay.off_fb() + i * T + g], upd = tab[lp.lay.off_upd() + i * T + g];
                const double sync = tab[lp.lay.off_sync() + (size_t)i * lp.lay.R + d];
                if (dist == 0) {                                  // the last stage sends nothing
                    best.sum = fb; best.mx = fb; best.sy = sync; best.up = upd;
                } else {
                    double best_v = make_inf();
#pragma unroll
                    for (uint32_t g2 = 0; g2 < TM; ++g2) {
                        if (d2v[g2] == DP_NONE || !(n[g2].sum < make_inf())) continue;
                        const double t = add_rn(fb, tab[lp.lay.off_c2x() + (size_t)d2v[g2] * lp.lay.R + d]);
                        DpVal c;
                        c.sum = add_rn(t, n[g2].sum);
                        c.mx = dmax(t, n[g2].mx);
                        c.sy = dmax(sync, n[g2].sy);
                        c.up = dmax(upd, n[g2].up);
                        const double val = add_rn(add_rn(add_rn(c.sum, mul_rn(nb, c.mx)), c.sy), c.up);
                        if (pick == DP_NONE || val < best_v) { best = c; best_v = val; pick = (uint8_t)g2; }
                    }
                }
            }
            cur[e0 + g * S] = best;
            choice[e0 + g * S] = pick;
        }
    }
}

template <uint32_t TM>
__global__ void __launch_bounds__(DP_THREADS, TM <= 4 ? 3 : 2) dp_level_vec_kernel(const __grid_constant__ DpLevelParams lp) {
    extern __shared__ uint32_t s_vt[];                       // the problem's rank tables
    __shared__ DpProblem pb;
    __shared__ uint32_t s_lo;
    const uint32_t tid = threadIdx.x;
    uint32_t which = 0;
    // the problem whose blocks include this one: a search with DP_THREADS probes per round instead of two, so that
    // a block waits for one or two loads, not for a chain of them
    {
        uint32_t lo = 0, n = lp.n_active;                    // invariant: prefix[lo] <= block < prefix[lo + n]
        while (n > 1) {
            const uint32_t step = (n + DP_THREADS - 1) / DP_THREADS;
            const uint32_t a = lo + tid * step, b = a + step < lo + n ? a + step : lo + n;
            if (a < lo + n && lp.blk_prefix[a] <= blockIdx.x && blockIdx.x < lp.blk_prefix[b]) s_lo = a;
            __syncthreads();
            const uint32_t got = s_lo;
            __syncthreads();
            n = got + step < lo + n ? step : lo + n - got;
            lo = got;
        }
        which = lo;
    }
    const uint32_t first = (blockIdx.x - lp.blk_prefix[which]) * (DP_THREADS * lp.per_thread);
    {
        const DpProblem* src = lp.problems + which;
        for (uint32_t x = tid; x < sizeof(DpProblem) / 4; x += DP_THREADS)
            reinterpret_cast<uint32_t*>(&pb)[x] = reinterpret_cast<const uint32_t*>(src)[x];
    }
    __syncthreads();
    for (uint32_t x = tid; x < pb.vt_len; x += DP_THREADS) s_vt[x] = lp.vtabs[pb.vt_lo + x];
    __syncthreads();
    // offsets into the rank tables count from the start of all tables: the staged copy is addressed the same way
    const uint32_t* const vtabs = s_vt - pb.vt_lo;
    dp_vec_level<TM>(lp, pb, vtabs, lp.dist, first, lp.per_thread);
}

// Small problems: a block takes one problem through all its stages, from the last to the first, with a barrier
// between stages (a stage reads only what the same block wrote for the stage after it): one launch per batch
// instead of one per stage.
template <uint32_t TM>
__global__ void __launch_bounds__(DP_THREADS, TM <= 4 ? 3 : 2) dp_problem_kernel(const __grid_constant__ DpLevelParams lp) {
    extern __shared__ uint32_t s_vt[];                       // the problem's rank tables
    __shared__ DpProblem pb;
    const uint32_t tid = threadIdx.x;
    {
        const DpProblem* src = lp.problems + blockIdx.x;
        for (uint32_t x = tid; x < sizeof(DpProblem) / 4; x += DP_THREADS)
            reinterpret_cast<uint32_t*>(&pb)[x] = reinterpret_cast<const uint32_t*>(src)[x];
    }
    __syncthreads();
    for (uint32_t x = tid; x < pb.vt_len; x += DP_THREADS) s_vt[x] = lp.vtabs[pb.vt_lo + x];
    __syncthreads();
    const uint32_t* const vtabs = s_vt - pb.vt_lo;
    for (uint32_t dist = 0; dist < pb.P; ++dist) {
        const uint32_t budget = pb.P - dist;                 // stage i = P - 1 - dist has at most i + 1 stages behind it
        uint32_t vectors = 0;
        for (uint32_t zp = 0; zp < pb.nz; ++zp) {
            uint32_t wz = 1;
            if (pb.rank_off[zp] != DP_DENSE) {
                const uint32_t* row0 = vtabs + pb.rank_off[zp];
                wz = row0[budget] - row0[budget - 1];
            }
            vectors += wz;
        }
        dp_vec_level<TM>(lp, pb, vtabs, dist, 0, (vectors + DP_THREADS - 1) / DP_THREADS);
        __syncthreads();
    }
}

// Stage 0 and the walk through the kept choices: one thread per problem.
struct DpFinishParams {
    const unsigned char* blob;
    const uint16_t* avail;
    SpaceDesc sp;
    const DpProblem* problems;
    const double* tabs;
    const uint32_t* vtabs;
    const DpVal* val[2];
    const uint8_t* choice;
    DpResult* results;               // indexed by problem index
    DpTabLayout lay;
    uint32_t n_problems, T;
};

__global__ void __launch_bounds__(128) dp_finish_kernel(const __grid_constant__ DpFinishParams fp) {
    const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= fp.n_problems) return;
    const DpProblem& pb = fp.problems[x];
    DpResult& out = fp.results[pb.index];
    const uint32_t T = fp.T, P = pb.P;
    const double* tab = fp.tabs + (size_t)pb.config * fp.lay.stride();
    const uint32_t* okv = reinterpret_cast<const uint32_t*>(tab + fp.lay.off_ok());
    const double nb = (double)*reinterpret_cast<const uint64_t*>(tab + fp.lay.off_nb());
    const DpVal* lvl0 = fp.val[(P - 1) & 1] + pb.val_off;
    double best_v = make_inf();
    uint32_t g = DP_NONE, zp = 0, entry = 0;
    for (uint32_t g0 = 0; g0 < T; ++g0) {                    // stage 0 by first fit from the first zone of the order
        if (!((okv[0] >> g0) & 1u)) continue;
        const uint32_t p = pb.cap[0][g0] >= 1 ? 0u : pb.first_later[0][g0];
        if (p == DP_NONE) continue;
        const uint32_t e = pb.zp_base[p] + g0 * pb.S[p] + pb.first_idx[p][g0];
        const DpVal v = lvl0[e];
        if (!(v.sum < make_inf())) continue;
        const double val = add_rn(add_rn(add_rn(v.sum, mul_rn(nb, v.mx)), v.sy), v.up);
        if (g == DP_NONE || val < best_v) { best_v = val; g = g0; zp = p; entry = e; }
    }
    out.value = best_v;
    if (g == DP_NONE) return;
    const Config k = config_of(fp.sp, pb.config);
    sailor_run runs[SAILOR_P_MAX];
    uint32_t n_runs = 0;
    for (uint32_t i = 0; i < P; ++i) {
        const uint8_t z = pb.zone[zp];
        out.type[i] = (uint8_t)g;
        out.zone[i] = z;
        if (n_runs && runs[n_runs - 1].type == g && runs[n_runs - 1].zone == z) runs[n_runs - 1].n_stages++;
        else {
            runs[n_runs].type = (uint8_t)g; runs[n_runs].zone = z;
            runs[n_runs].tp_idx = (uint8_t)k.tpi; runs[n_runs].n_stages = 1;
            ++n_runs;
        }
        if (i + 1 == P) break;
        const uint8_t g2 = fp.choice[pb.choice_off + (size_t)i * pb.n_lvl + entry];
        const uint32_t ui = (entry - pb.zp_base[zp]) % pb.S[zp];
        uint32_t u[SAILOR_T_MAX];
        dp_counts(pb, fp.vtabs, zp, T, ui, u, P);
        const DpMove mv = dp_move(pb, fp.vtabs, T, zp, ui, u, g2);
        g = g2; zp = mv.zp; entry = mv.entry;
    }
    // the plan written out, through the simulator (Sec. 4.3): what a caller compares with a constraint
    TabView v;
    v.bind(fp.blob, fp.blob);
    uint32_t cnt[R_MAX];
    const SimOut so = simulate_runs(v, fp.avail, P, n_runs, k.D, k.mi, k.rc, runs, SAILOR_P_MAX, cnt, 1);
    out.t_iter = so.t_iter;
    out.cost = so.cost;
    out.peak_mem = so.peak_mem;
    out.status = so.status;
}

// The k best problems by (value, problem index), then the simulator's figures for their plans.
struct DpSelectParams {
    const DpResult* results;
    sailor_dp_result* out;           // [k] device
    unsigned long long* counters;    // [0] problems with a plan, [1] number written to out, [2] plans over the constraint
    SpaceDesc sp;
    uint32_t n_problems, n_orders, k;
    double budget, min_rate;         // <= 0: none
};

constexpr int DP_SELECT_THREADS = 512;

__global__ void __launch_bounds__(DP_SELECT_THREADS) dp_select_kernel(const __grid_constant__ DpSelectParams sp) {
    __shared__ Hit s_hits[DP_SELECT_THREADS / 32][SAILOR_K_MAX];
    __shared__ uint32_t s_n;
    __shared__ unsigned long long s_solved, s_over;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = DP_SELECT_THREADS / 32;
    if (tid == 0) { s_solved = 0; s_over = 0; }
    __syncthreads();
    WarpTopK top;
    top.init();
    uint32_t solved = 0, over = 0;
    for (uint32_t base = warp * 32; base < sp.n_problems; base += nw * 32) {
        const uint32_t j = base + lane;
        const double v = j < sp.n_problems ? sp.results[j].value : make_inf();
        bool have = v < make_inf();
        solved += have;
        if (have) {                                           // the planner keeps a plan only within the constraint
            const DpResult& r = sp.results[j];
            const bool out_of = (sp.budget > 0.0 && r.cost > sp.budget) || (sp.min_rate > 0.0 && 1.0 / r.t_iter < sp.min_rate);
            over += out_of;
            have = !out_of;
        }
        const bool want = have && v <= top.thr_score;
        if (__any_sync(FULL, want)) top.offer(want, v, j, sp.k, lane);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        solved += __shfl_xor_sync(FULL, solved, o);
        over += __shfl_xor_sync(FULL, over, o);
    }
    if (lane == 0 && solved) atomicAdd(&s_solved, (unsigned long long)solved);
    if (lane == 0 && over) atomicAdd(&s_over, (unsigned long long)over);
    s_hits[warp][lane].score = top.score;
    s_hits[warp][lane].flat = top.flat;
    __syncthreads();
    for (uint32_t step = 1; step < nw; step <<= 1) {
        if ((warp & (2 * step - 1)) == 0 && warp + step < nw) {
            top.merge_sorted(s_hits[warp + step][lane].score, s_hits[warp + step][lane].flat, sp.k, lane);
            s_hits[warp][lane].score = top.score;
            s_hits[warp][lane].flat = top.flat;
        }
        __syncthreads();
    }
    if (warp == 0) {
        const uint32_t n = __popc(__ballot_sync(FULL, lane < sp.k && top.flat != ~0ull));
        if (lane == 0) {
            s_n = n;
            sp.counters[0] = s_solved;
            sp.counters[1] = n;
            sp.counters[2] = s_over;
        }
    }
    __syncthreads();
    for (uint32_t j = warp; j < s_n; j += nw) {
        if (lane != 0) continue;
        const uint32_t idx = (uint32_t)s_hits[0][j].flat;
        const DpResult& r = sp.results[idx];
        const uint32_t c = idx / sp.n_orders;
        const Config k = config_of(sp.sp, c);
        sailor_dp_result o;
        for (int q = 0; q < (int)sizeof(o); ++q) reinterpret_cast<unsigned char*>(&o)[q] = 0;
        o.config = c;
        o.order = idx % sp.n_orders;
        o.value = r.value;
        o.P = (uint8_t)k.P; o.mbs_idx = (uint8_t)k.mi; o.tp_idx = (uint8_t)k.tpi; o.rc = (uint8_t)k.rc; o.D = (uint16_t)k.D;
        for (uint32_t i = 0; i < k.P; ++i) {
            o.type[i] = r.type[i];
            o.zone[i] = r.zone[i];
        }
        o.t_iter = r.t_iter;
        o.cost = r.cost;
        o.peak_mem = r.peak_mem;
        o.status = r.status;
        sp.out[j] = o;
    }
}

}  // namespace sailor
