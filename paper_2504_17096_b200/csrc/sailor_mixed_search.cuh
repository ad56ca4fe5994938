// Search over plans whose stages mix GPU types among their replicas (Sailor Sec. 4.2.2, "Implementation": per
// stage, the resource combinations of different GPU types that give the stage its D replicas).
//
// A combination is a tuple of units per GPU type (see sailor.h); the host lists the combinations of every degree
// of the space once per call (descending lexicographic order) and the device looks them up.  A candidate is
// (P, mbs, rc, D) and one (zone, combination) per segment; one warp builds the candidate's record in shared memory
// from its flat index, evaluates it with simulate_mixed_plan (a lane per stage) and offers it to its top-k list, which
// here is a warp-uniform insertion.  Blocks leave their lists for mixed_finish_kernel, which merges them and writes
// the winners out with their records.
#pragma once

#include "sailor_mixed.cuh"
#include "sailor_plan_kernels.cuh"

namespace sailor {

constexpr uint32_t MIX_UNITS_MAX = 16;
static_assert(SAILOR_MIX_P_MAX % 32 == 0, "every lane writes SAILOR_MIX_P_MAX / 32 stages of the record");

struct MixedSpaceDesc {
    uint32_t n_p, n_mbs, n_rc, n_d, seg_max, granularity;
    uint8_t p_values[SAILOR_NP_MAX];
    uint8_t mbs_idx[SAILOR_MBS_MAX];
    uint8_t rc_values[2];
    uint8_t tp_idx_of_type[SAILOR_T_MAX];
    uint16_t d_values[SAILOR_ND_MAX];
    uint32_t n_comb[SAILOR_ND_MAX];          // combinations of each degree of d_values
    uint32_t comb_off[SAILOR_ND_MAX];        // where they start in the table
};

__host__ __device__ inline uint32_t mixed_units(uint32_t granularity, uint32_t D) {
    return (granularity >= 1 && D % granularity == 0) ? granularity : D;
}

// Configuration c = ((p * n_mbs + mbs) * n_rc + rc) * n_d + d (positions in the space's lists).
struct MixedConfig { uint32_t P, mi, rc, D, di, nseg, per_unit; };   // per_unit: replicas in one unit of a combination

__host__ __device__ inline MixedConfig mixed_config_of(const MixedSpaceDesc& s, uint32_t c) {
    MixedConfig k;
    uint32_t x = c;
    k.di = x % s.n_d; x /= s.n_d;
    const uint32_t ri = x % s.n_rc; x /= s.n_rc;
    const uint32_t mi = x % s.n_mbs; x /= s.n_mbs;
    k.P = s.p_values[x];
    k.mi = s.mbs_idx[mi];
    k.rc = s.rc_values[ri];
    k.D = s.d_values[k.di];
    k.nseg = k.P < s.seg_max ? k.P : s.seg_max;
    k.per_unit = k.D / mixed_units(s.granularity, k.D);
    return k;
}

// Stage i of the candidate whose segment digits are `digit` (zone * n_comb + combination): its record.
// `combs` holds one 64-bit word per combination, byte g = units on type g.
__host__ __device__ inline void mixed_build_stage(const MixedSpaceDesc& s, const MixedConfig& k, uint32_t T,
                                                  const uint64_t* combs, const uint32_t* digit, uint32_t i,
                                                  sailor_mixed_stage* out) {
    const uint32_t n_comb = s.n_comb[k.di];
    const uint32_t dg = digit[i * k.nseg / k.P], zone = dg / n_comb;       // a digit is below Z * n_comb < 2^32
    const uint64_t word = combs[s.comb_off[k.di] + (dg - zone * n_comb)];
    // the stage as five 32-bit words (little-endian fields): zone | n_groups << 8, then type | tp_idx << 8 | count << 16
    // per group; the non-empty types in ascending order take the groups
    uint32_t gw[SAILOR_MIX_GROUPS_MAX] = {0, 0, 0, 0}, n_groups = 0;
    for (uint32_t g = 0; g < T; ++g) {
        const uint32_t units = (uint32_t)(word >> (8 * g)) & 0xffu;
        if (!units || n_groups >= SAILOR_MIX_GROUPS_MAX) continue;
        const uint32_t grp = g | (uint32_t)s.tp_idx_of_type[g] << 8 | (units * k.per_unit & 0xffffu) << 16;
        gw[0] = n_groups == 0 ? grp : gw[0];
        gw[1] = n_groups == 1 ? grp : gw[1];
        gw[2] = n_groups == 2 ? grp : gw[2];
        gw[3] = n_groups == 3 ? grp : gw[3];
        n_groups++;
    }
    static_assert(sizeof(sailor_mixed_stage) == 20 && SAILOR_MIX_GROUPS_MAX == 4, "five words a stage");
    uint32_t* w = reinterpret_cast<uint32_t*>(out);
    w[0] = (zone & 0xffu) | n_groups << 8;
    w[1] = gw[0]; w[2] = gw[1]; w[3] = gw[2]; w[4] = gw[3];
}

struct MixedSearchParams {
    const unsigned char* blob;
    const uint16_t* avail;
    const uint64_t* cfg_flat_base;       // [n_config + 1]
    const uint64_t* combs;
    Hit* partial;                        // [grid][SAILOR_K_MAX]
    unsigned long long* counters;        // total, invalid, oom, over_avail, over_constraint, feasible, min cost bits, error
    sailor_mixed_result* results;        // [k] device
    MixedSpaceDesc sp;
    uint32_t n_config, k, obj, n_partial;
    uint64_t n_total;
    double budget, min_rate;             // <= 0: none
};

constexpr int MIXS_THREADS = 256;
constexpr int MIXS_WARPS = MIXS_THREADS / 32;

// The record of candidate `flat` into `plan` (shared memory, one per warp), by all lanes of the warp.  WHOLE: the
// stages past the last are zeroed as well (a record that leaves the device); the evaluation reads the first P only.
// The configuration of a warp's previous candidate (a warp's candidates are a grid stride apart and mostly stay
// inside one configuration): tried first, decoded anew only when the index has left it.
struct MixedCursor {
    uint32_t cfg = ~0u;
    uint64_t lo = 1, hi = 0;             // flat indices [lo, hi) of the configuration
    MixedConfig k;
};

template <bool WHOLE>
__device__ __forceinline__ void mixed_candidate(const MixedSearchParams& mp, uint32_t T, uint32_t Z, uint64_t flat,
                                                sailor_mixed_plan* plan, uint32_t lane, MixedCursor& cur) {
    if (!(cur.lo <= flat && flat < cur.hi)) {
        uint32_t lo = 0, hi = mp.n_config;                   // the configuration whose block holds the index
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (mp.cfg_flat_base[mid] <= flat) lo = mid; else hi = mid;
        }
        cur.cfg = lo;
        cur.lo = mp.cfg_flat_base[lo];
        cur.hi = mp.cfg_flat_base[lo + 1];
        cur.k = mixed_config_of(mp.sp, lo);
    }
    const MixedConfig& k = cur.k;
    const uint64_t radix = (uint64_t)Z * mp.sp.n_comb[k.di];
    uint64_t rem = flat - cur.lo;
    uint32_t digit[SAILOR_SEG_MAX] = {0, 0, 0, 0};
    if ((rem >> 32) == 0) {                                  // the usual case: 32-bit divisions
        uint32_t r32 = (uint32_t)rem;
        const uint32_t rx = (uint32_t)radix;
        for (uint32_t s = k.nseg; s-- > 0;) { const uint32_t q = r32 / rx; digit[s] = r32 - q * rx; r32 = q; }
    } else {
        for (uint32_t s = k.nseg; s-- > 0;) { digit[s] = (uint32_t)(rem % radix); rem /= radix; }
    }
    if (lane == 0) {
        plan->P = (uint8_t)k.P; plan->mbs_idx = (uint8_t)k.mi; plan->rc = (uint8_t)k.rc; plan->_pad = 0;
        plan->D = (uint16_t)k.D; plan->_pad2 = 0;
    }
    for (uint32_t i = lane; i < (WHOLE ? (uint32_t)SAILOR_MIX_P_MAX : k.P); i += 32) {
        if (i < k.P) mixed_build_stage(mp.sp, k, T, mp.combs, digit, i, &plan->stage[i]);
        else {                                                 // stages past the last are all zero, as the host decoder leaves them
            uint32_t* z = reinterpret_cast<uint32_t*>(&plan->stage[i]);
            for (uint32_t x = 0; x < sizeof(sailor_mixed_stage) / 4; ++x) z[x] = 0;
        }
    }
    __syncwarp();
}

// DEEP: the space has pipelines of more than 32 stages (the evaluation then goes through the tiled variant).
template <bool DEEP>
__global__ void __launch_bounds__(MIXS_THREADS, 2) plan_mixed_kernel(const __grid_constant__ MixedSearchParams mp) {
    extern __shared__ __align__(16) unsigned char dyn[];      // static tables, then per-warp counters, then per-warp records
    __shared__ uint64_t mbar;
    __shared__ Hit s_hits[MIXS_WARPS][SAILOR_K_MAX];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t static_bytes = reinterpret_cast<const TabHdr*>(mp.blob)->static_bytes;
    if (!bulk_load(dyn, mp.blob, static_bytes, &mbar)) {
        if (tid == 0) atomicExch(&mp.counters[7], 1ull);
        for (uint32_t x = tid; x < static_bytes / 16; x += MIXS_THREADS)
            reinterpret_cast<uint4*>(dyn)[x] = reinterpret_cast<const uint4*>(mp.blob)[x];
        __syncthreads();
    }
    TabView v;
    v.bind(dyn, mp.blob);
    const uint32_t T = v.h->T, Z = v.h->Z, R = v.h->R;
    unsigned long long* cnt = reinterpret_cast<unsigned long long*>(dyn + static_bytes) + (size_t)warp * R;
    sailor_mixed_plan* plan = reinterpret_cast<sailor_mixed_plan*>(dyn + static_bytes + sizeof(unsigned long long) * MIXS_WARPS * R) + warp;
    WarpTopK top;
    top.init();
    unsigned long long n_class[6] = {0, 0, 0, 0, 0, 0};
    double min_cost = make_inf();
    const uint64_t stride = (uint64_t)gridDim.x * MIXS_WARPS;
    MixedCursor cur;                                           // configuration of this warp's previous candidate
    for (uint64_t flat = (uint64_t)blockIdx.x * MIXS_WARPS + warp; flat < mp.n_total; flat += stride) {
        mixed_candidate<false>(mp, T, Z, flat, plan, lane, cur);
        const SimOut o = DEEP ? simulate_mixed_plan(v, mp.avail, *plan, cnt, lane) : simulate_mixed_warp(v, mp.avail, *plan, cnt, lane);
        __syncwarp();                                          // the record and the counters are reused by the next candidate
        // every candidate falls in exactly one class: invalid, out of memory, over availability, over the constraint, feasible
        n_class[0]++;
        if (o.status & (SAILOR_ST_INVALID | SAILOR_ST_BAD_RECORD)) { n_class[1]++; continue; }
        if (o.status & SAILOR_ST_OOM) { n_class[2]++; continue; }
        if (o.status & SAILOR_ST_OVER_AVAIL) { n_class[3]++; continue; }
        bool over = false;
        if (mp.budget > 0.0 && o.cost > mp.budget) over = true;
        if (mp.min_rate > 0.0 && 1.0 / o.t_iter < mp.min_rate) over = true;
        if (over) { n_class[4]++; continue; }
        n_class[5]++;
        min_cost = o.cost < min_cost ? o.cost : min_cost;
        const double score = mp.obj == SAILOR_OBJ_MAX_THROUGHPUT ? o.t_iter : mp.obj == SAILOR_OBJ_MIN_COST ? o.cost : mul_rn(o.t_iter, o.cost);
        top.insert(score, flat, mp.k, lane);                   // every lane holds the same candidate
    }
    if (lane == 0) {
        for (int j = 0; j < 6; ++j)
            if (n_class[j]) atomicAdd(&mp.counters[j], n_class[j]);
        atomicMin(&mp.counters[6], (unsigned long long)__double_as_longlong(min_cost));
    }
    s_hits[warp][lane].score = top.score;
    s_hits[warp][lane].flat = top.flat;
    __syncthreads();
    if (warp == 0) {
        for (uint32_t w = 1; w < MIXS_WARPS; ++w) {
            if (s_hits[w][0].flat == ~0ull) continue;
            top.merge_sorted(s_hits[w][lane].score, s_hits[w][lane].flat, mp.k, lane);
        }
        mp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].score = lane < mp.k ? top.score : make_inf();
        mp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].flat = lane < mp.k ? top.flat : ~0ull;
    }
}

// Merge the blocks' lists; the winners are built and simulated again for the result records (a warp each).
__global__ void __launch_bounds__(MIXS_THREADS) mixed_finish_kernel(const __grid_constant__ MixedSearchParams mp) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ uint64_t mbar;
    __shared__ Hit s_hits[MIXS_WARPS][SAILOR_K_MAX];
    __shared__ uint32_t s_n;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t static_bytes = reinterpret_cast<const TabHdr*>(mp.blob)->static_bytes;
    if (!bulk_load(dyn, mp.blob, static_bytes, &mbar)) {
        if (tid == 0) atomicExch(&mp.counters[7], 1ull);
        for (uint32_t x = tid; x < static_bytes / 16; x += MIXS_THREADS)
            reinterpret_cast<uint4*>(dyn)[x] = reinterpret_cast<const uint4*>(mp.blob)[x];
        __syncthreads();
    }
    TabView v;
    v.bind(dyn, mp.blob);
    const uint32_t T = v.h->T, Z = v.h->Z, R = v.h->R;
    unsigned long long* cnt = reinterpret_cast<unsigned long long*>(dyn + static_bytes) + (size_t)warp * R;
    sailor_mixed_plan* plan = reinterpret_cast<sailor_mixed_plan*>(dyn + static_bytes + sizeof(unsigned long long) * MIXS_WARPS * R) + warp;
    WarpTopK top;
    top.init();
    for (uint32_t b = warp; b < mp.n_partial; b += MIXS_WARPS) {
        const Hit hme = mp.partial[(size_t)b * SAILOR_K_MAX + lane];
        if (__shfl_sync(FULL, hme.flat, 0) == ~0ull) continue;   // an empty list
        top.merge_sorted(hme.score, hme.flat, mp.k, lane);
    }
    s_hits[warp][lane].score = top.score;
    s_hits[warp][lane].flat = top.flat;
    __syncthreads();
    for (uint32_t step = 1; step < MIXS_WARPS; step <<= 1) {
        if ((warp & (2 * step - 1)) == 0 && warp + step < MIXS_WARPS) {
            top.merge_sorted(s_hits[warp + step][lane].score, s_hits[warp + step][lane].flat, mp.k, lane);
            s_hits[warp][lane].score = top.score;
            s_hits[warp][lane].flat = top.flat;
        }
        __syncthreads();
    }
    if (warp == 0) {
        const uint32_t n = __popc(__ballot_sync(FULL, lane < mp.k && top.flat != ~0ull));
        if (lane == 0) s_n = n;
    }
    __syncthreads();
    for (uint32_t j = warp; j < s_n; j += MIXS_WARPS) {
        const uint64_t flat = s_hits[0][j].flat;
        MixedCursor cur;
        mixed_candidate<true>(mp, T, Z, flat, plan, lane, cur);
        const SimOut o = simulate_mixed_plan(v, mp.avail, *plan, cnt, lane);
        __syncwarp();
        sailor_mixed_result* r = mp.results + j;
        if (lane == 0) {
            r->flat = flat; r->t_iter = o.t_iter; r->cost = o.cost; r->peak_mem = o.peak_mem;
            r->score = s_hits[0][j].score; r->status = o.status; r->_pad = 0;
        }
        // the record, word by word
        const uint64_t* src = reinterpret_cast<const uint64_t*>(plan);
        uint64_t* dst = reinterpret_cast<uint64_t*>(&r->plan);
        for (uint32_t x = lane; x < sizeof(sailor_mixed_plan) / 8; x += 32) dst[x] = src[x];
        __syncwarp();
    }
    if (tid == 0) mp.counters[8] = s_n;
}

}  // namespace sailor
