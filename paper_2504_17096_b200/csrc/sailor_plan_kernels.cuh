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
#ifndef PLAN_DIGITS_PER_STEP
#define PLAN_DIGITS_PER_STEP 4      // candidates evaluated side by side per thread (independent chains)
#endif
#ifndef PLAN_MIN_BLOCKS
#define PLAN_MIN_BLOCKS 2
#endif
#ifndef PLAN_SCREEN_BLOCKS
#define PLAN_SCREEN_BLOCKS 3        // resident blocks per SM the screened kernels are compiled for (binary32 state is half as wide)
#endif
constexpr unsigned FULL = 0xffffffffu;
constexpr uint32_t WAIT_LIMIT = 1u << 22;   // bound of every spin-wait in this file

struct alignas(16) Hit {
    double score;
    uint64_t flat;
};

struct Ctrl {                       // one per context, device memory
    unsigned int work_counter;      // next chunk to hand out (starts at zero in every launch)
    unsigned int blocks_done;       // blocks of the running launch that have handed in their list
    unsigned long long stats[7];    // total, invalid, oom, over_avail, over_constraint, feasible, pruned_tp
    unsigned int wave_chunks;       // chunks of the current wave (searches in degree order)
    unsigned int n_cfg_evaluated;   // configurations selected by the waves so far
    unsigned long long min_cost_bits;   // min C_iter over feasible candidates, as ordered bits
    unsigned long long thr_bits;    // a score no candidate of the final top-k exceeds (ordered bits): the best k-th
                                    // best any warp has seen so far; lets all other warps skip what cannot matter
    double budget;                  // written by the cheapest-plan pass for the next pass
    unsigned int error;             // non-zero: a kernel gave up during this call (bounded wait ran out)
    unsigned int n_found;
};

// What a pass leaves for the host (one device-to-host copy: the counters, then the k records).  The block that
// finishes a pass writes it and then puts the live counters back to their starting values, so that the next pass
// or the next call needs no clearing from the host.
struct PlanOut {
    Ctrl ctrl;
    sailor_result results[SAILOR_K_MAX];
};

constexpr unsigned long long COST_BITS_START = 0x7ff0000000000000ull;   // +inf: above every cost

struct PlanParams {
    const unsigned char* blob;
    uint16_t avail[R_MAX];             // the availability snapshot rides in the launch parameters: a search needs no
                                       // copy of its own before it, and 128 bytes are well within the parameter space
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
    uint32_t live_mode;                // cfg_chunk_start counts only chunks of prefixes made of usable digits
    uint32_t min_tp_only;              // drop plans that also fit with a smaller tensor-parallel degree (H2)
    uint32_t carry_lists;              // a block starts from the list it left in `partial` (waves of one search)
    const uint32_t* chunk_hi_dev;      // non-null: chunks [0, *chunk_hi_dev) instead of [chunk_lo, chunk_hi)
    unsigned long long* cfg_best;      // non-null: [n_config] best feasible score per configuration (ordered bits)
    PlanOut* out;                      // where the block that finishes the pass leaves the results
    uint32_t finish;                   // this launch ends a pass: its last block merges the lists and writes `out`
    double next_budget_factor;         // > 0: the finishing block writes ctrl->budget = factor * best cost (next pass)
    uint32_t cost_only;                // the pass only looks for the cheapest feasible cost (no lists, no result records)
    uint32_t screen;                   // candidates are first evaluated in binary32 (SCREEN kernels): sizes the shared tables
    const uint4* cfg_cache;            // non-null: the per-configuration tables, built once per space (cfg_cache_kernel)
    uint32_t cache_head16, cache_arr16;    // 16-byte words of a cached record: CfgShared head, then the arrays
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
    // Returns false when the candidate is not better than the current k-th (warp-uniform).
    __device__ __forceinline__ bool insert(double s, uint64_t f, uint32_t k, uint32_t lane) {
        if (!(s < thr_score || (s == thr_score && f < thr_flat))) return false;   // warp-uniform
        const bool before = (score < s) || (score == s && flat < f);
        const uint32_t pos = __popc(__ballot_sync(FULL, before));           // sorted: a prefix of lanes
        const double ps = __shfl_up_sync(FULL, score, 1);
        const uint64_t pf = __shfl_up_sync(FULL, flat, 1);
        if (lane > pos) { score = ps; flat = pf; }
        else if (lane == pos) { score = s; flat = f; }
        thr_score = __shfl_sync(FULL, score, k - 1);
        thr_flat = __shfl_sync(FULL, flat, k - 1);
        return true;
    }
    // Merge another ascending list of 32 (lane j passes its j-th element; empty slots are
    // (+inf, ~0)) into this one, keeping the 32 smallest of the union: min(a[j], b[31-j]) is a
    // bitonic sequence holding exactly those, and five compare-exchange stages sort it.
    __device__ __forceinline__ void merge_sorted(double bs, uint64_t bf, uint32_t k, uint32_t lane) {
        const double rs = __shfl_sync(FULL, bs, 31 - lane);
        const uint64_t rf = __shfl_sync(FULL, bf, 31 - lane);
        if (rs < score || (rs == score && rf < flat)) { score = rs; flat = rf; }
#pragma unroll
        for (int stride = 16; stride; stride >>= 1) {
            const double os = __shfl_xor_sync(FULL, score, stride);
            const uint64_t of = __shfl_xor_sync(FULL, flat, stride);
            const bool other_less = os < score || (os == score && of < flat);
            const bool upper = lane & stride;
            if (other_less != upper) { score = os; flat = of; }     // lower lane keeps the smaller, upper the larger
        }
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
//
// Inside one segment all stages share (type, zone, tp), so their per-microbatch times take at
// most four distinct values, in stage order: stage 0 (embedding), stages with one extra block,
// plain stages, the final stage (head, sends nothing).  A segment is therefore stored as four
// (count, value[digit]) runs; adding `count` copies of `value` one after the other is the same
// sequence of additions as walking the stages.  The last stage of a non-final segment sends to
// the next segment, so its time depends on two digits and is kept apart (fb_last + c2x).
constexpr int N_RUNS = 4;
constexpr uint32_t PLAN_PAD = PLAN_DIGITS_PER_STEP - 1;   // table entries past the last digit that a step may read

struct alignas(16) SegRec {                  // one per (segment, digit); 64 bytes, read as broadcasts
    double v[N_RUNS];            // t_i of each run (f + b + 2c with the next stage on the same digit)
    double tmax;                 // max of v[] over the non-empty runs
    double sync;                 // max all-reduce time over the segment's stages
    double upd;                  // max update time over the segment's stages
    double rate;                 // D * tp * price per second of one stage
};

// The binary32 screen (optional search mode): every candidate is first evaluated in binary32 from rounded copies of
// the tables; an item (a prefix with all its last digits) is evaluated again in binary64, exactly as without the
// screen, only when its best binary32 score comes within SCREEN_BAND of the score a candidate must beat to enter
// the top-k, or its cheapest binary32 cost within SCREEN_BAND of the cheapest cost known.  A binary32 evaluation
// rounds each table entry once (2^-24) and adds at most P + 4 positive terms (each addition 2^-24), multiplies
// twice and, for throughput per cost, once more: a relative error below (P + 12) * 2^-24 < 7e-6 for P <= 96 in time
// and cost, below 1.4e-5 in their product.  The band is 1e-4, so every candidate whose exact score could enter the
// list (or whose exact cost could be the cheapest) is looked at exactly: lists, counts and statistics are the
// exact search's, bit for bit.
constexpr double SCREEN_BAND = 1e-4;

struct alignas(16) SegRec32 {                // SegRec rounded to binary32; 32 bytes
    float v[N_RUNS];
    float tmax, sync, upd, rate;
};

struct alignas(16) CfgShared {
    // scalars (written by thread 0 / the build, read by all)
    Config cfg;
    uint32_t valid;              // gbs % (D*mbs) == 0 and heads % tp == 0
    uint32_t packed;             // prefixes are enumerated over the usable digits of each segment only
    uint32_t g_cnt[SAILOR_SEG_MAX];       // usable digits (valid type, fits in memory) per segment
    uint32_t g_magic[SAILOR_SEG_MAX];     // floor(2^32 / g_cnt) + 1, for division by g_cnt
    uint64_t live_items;         // product of g_cnt over the prefix segments
    uint8_t good_list[SAILOR_SEG_MAX][R_MAX];   // the usable digits of each segment, ascending
    uint32_t seg_a[SAILOR_SEG_MAX + 1];   // first stage of each segment; seg_a[nseg] = P
    uint32_t need[SAILOR_SEG_MAX];        // GPUs a segment takes of its digit: D * tp * stages
    uint32_t n_run[SAILOR_SEG_MAX][N_RUNS];   // stages in each run (without a non-final segment's last stage)
    double ar_steps, ar_coef;    // 2(D-1) and 2(D-1)/D of the ring all-reduce
    uint64_t n_b;
    uint64_t n_items;            // R^(nseg-1)
    uint64_t invalid_mask;       // digit d: tp > gpus_per_node[type(d)]
    uint64_t oom_mask[SAILOR_SEG_MAX];    // digit d: some stage of the segment does not fit type(d)
    uint32_t n_lower;            // smaller tensor-parallel degrees of the space that the model accepts (min_tp_only)
    uint32_t lower_tpi[SAILOR_TP_MAX];    // their tp indices
    uint64_t lower_fit[SAILOR_TP_MAX][SAILOR_SEG_MAX];   // digit d: every stage of the segment fits at that degree
    uint64_t flat_base;          // flat index of the configuration's first candidate
    uint64_t _pad_head;
    // ---- everything above depends on the configuration and the context only, not on availability: it is what a
    // ---- cached record holds (with the arrays rec .. fb_last); everything below belongs to the block or the snapshot
    alignas(16) uint64_t avail_last;     // digit d: need[last] <= avail[d]
    uint32_t magic;              // floor(2^32 / R) + 1: x / R == umulhi(x, magic) for x < 2^26
    uint32_t cur_config;
    uint32_t next_chunk, batch_len;
    unsigned long long oom_stage[SAILOR_P_MAX];   // per stage: bit 8 j + g set when the stage does not fit type g
                                                  // at this configuration's degree (j = 0) or at lower_tpi[j - 1]
    uint64_t params[SAILOR_P_MAX];
    unsigned long long stat[7];
    unsigned long long thr_bits;     // the block's copy of Ctrl::thr_bits, lowered by its own warps as their lists fill
    unsigned long long minc_bits;    // screened search: the cheapest exact cost the block's warps have seen (ordered bits)
    uint64_t mbar;
};

struct CfgArrays {               // pointers into dynamic shared memory
    SegRec* rec;                 // [SEG_MAX][R]
    double* c2x;                 // [R][R]   2 * message time, index [next digit][this digit]
    double* commx;               // [R][Z]   transfer cost of one boundary, index [next digit][this zone]
    double* fb_last;             // [SEG_MAX][T]  f+b of a segment's last stage, per type
    double *fb, *uu;             // [P][T]   build scratch: f+b (+f if rc), update
    uint32_t* availv;            // [R]
    uint32_t* tz;                // [R]      type | zone << 8 of a digit
    uint32_t* chunk_tab;         // [n_config + 1] copy of the chunk offsets (spaces of fewer than PLAN_CFG_SMEM configurations)
    SegRec32* rec32;             // screened search: rec, c2x, commx rounded to binary32 (same shapes and padding)
    float* c2x32;
    float* commx32;
};

constexpr uint32_t PLAN_CFG_SMEM = 4096;

__host__ __device__ inline size_t plan_screen_bytes(uint32_t T, uint32_t Z) {
    const size_t R = (size_t)T * Z;
    return sizeof(SegRec32) * (SAILOR_SEG_MAX * R + PLAN_PAD) + sizeof(float) * ((R + PLAN_PAD) * R + (R + PLAN_PAD) * Z) + 32;
}

__host__ __device__ inline size_t plan_smem_bytes(uint32_t static_bytes, uint32_t p_max, uint32_t T, uint32_t Z, uint32_t n_config,
                                                  bool screen = false) {
    const size_t R = (size_t)T * Z;
    size_t n = static_bytes;
    if (screen) n += plan_screen_bytes(T, Z);
    if (n_config < 4096) n += sizeof(uint32_t) * ((size_t)n_config + 1);
    n += sizeof(SegRec) * (SAILOR_SEG_MAX * R + PLAN_PAD);               // padding digits, see walk_fast
    n += sizeof(double) * ((R + PLAN_PAD) * R + (R + PLAN_PAD) * Z + (size_t)SAILOR_SEG_MAX * T + 2 * (size_t)p_max * T);
    n += sizeof(uint32_t) * 2 * R;
    return (n + 15) & ~(size_t)15;
}

// A cached configuration record: the head of CfgShared up to avail_last, then the arrays rec, c2x, commx, fb_last
// (with their padding entries), both in 16-byte words.
__host__ __device__ inline uint32_t cache_head16() { return (uint32_t)(offsetof(CfgShared, avail_last) / 16); }
__host__ __device__ inline uint32_t cache_arr16(uint32_t T, uint32_t Z) {
    const size_t R = (size_t)T * Z;
    const size_t bytes = sizeof(SegRec) * (SAILOR_SEG_MAX * R + PLAN_PAD) +
                         sizeof(double) * ((R + PLAN_PAD) * R + (R + PLAN_PAD) * Z + (size_t)SAILOR_SEG_MAX * T);
    return (uint32_t)((bytes + 15) / 16);
}

__device__ __forceinline__ void carve(unsigned char* dyn, uint32_t static_bytes, uint32_t p_max, uint32_t T,
                                      uint32_t Z, CfgArrays& a, uint32_t n_config = 0, bool screen = false) {
    const uint32_t R = T * Z;
    a.rec = reinterpret_cast<SegRec*>(dyn + static_bytes);           // static_bytes is a multiple of 16
    double* p = reinterpret_cast<double*>(a.rec + (size_t)SAILOR_SEG_MAX * R + PLAN_PAD);
    a.c2x = p;       p += (size_t)(R + PLAN_PAD) * R;
    a.commx = p;     p += (size_t)(R + PLAN_PAD) * Z;
    a.fb_last = p;   p += (size_t)SAILOR_SEG_MAX * T;
    a.fb = p;        p += (size_t)p_max * T;
    a.uu = p;        p += (size_t)p_max * T;
    a.availv = reinterpret_cast<uint32_t*>(p);
    a.tz = a.availv + R;
    a.chunk_tab = a.tz + R;
    a.rec32 = nullptr;
    a.c2x32 = a.commx32 = nullptr;
    if (screen) {
        uintptr_t at = reinterpret_cast<uintptr_t>(a.chunk_tab + (n_config < PLAN_CFG_SMEM ? n_config + 1 : 0));
        at = (at + 15) & ~(uintptr_t)15;
        a.rec32 = reinterpret_cast<SegRec32*>(at);
        a.c2x32 = reinterpret_cast<float*>(a.rec32 + (size_t)SAILOR_SEG_MAX * R + PLAN_PAD);
        a.commx32 = a.c2x32 + (size_t)(R + PLAN_PAD) * R;
    }
}

// The binary32 copies of the tables of the configuration just built or loaded.  Called by the whole block; ends
// synchronised.
__device__ __forceinline__ void round_config32(const CfgArrays& a, uint32_t R, uint32_t Z) {
    const uint32_t tid = threadIdx.x;
    for (uint32_t x = tid; x < SAILOR_SEG_MAX * R + PLAN_PAD; x += PLAN_THREADS) {
        const SegRec& r = a.rec[x];
        SegRec32 q;
        for (int j = 0; j < N_RUNS; ++j) q.v[j] = __double2float_rn(r.v[j]);
        q.tmax = __double2float_rn(r.tmax); q.sync = __double2float_rn(r.sync);
        q.upd = __double2float_rn(r.upd); q.rate = __double2float_rn(r.rate);
        a.rec32[x] = q;
    }
    for (uint32_t x = tid; x < (R + PLAN_PAD) * R; x += PLAN_THREADS) a.c2x32[x] = __double2float_rn(a.c2x[x]);
    for (uint32_t x = tid; x < (R + PLAN_PAD) * Z; x += PLAN_THREADS) a.commx32[x] = __double2float_rn(a.commx[x]);
    __syncthreads();
}

// Run of stage i: 0 = stage 0 with the embedding, 1 = one extra block, 2 = plain, 3 = final stage.
__device__ __forceinline__ uint32_t run_of(const TabHdr* h, uint32_t P, uint32_t extra, uint32_t i) {
    if (i == P - 1) return 3;
    if (i == 0 && h->has_embed) return 0;
    return i < extra ? 1 : 2;                              // extra = n_blocks % P
}

// Build the tables of configuration `c`.  Called by the whole block; ends synchronised.
__device__ void build_config(const PlanParams& pp, const TabView& v, CfgShared& cs, CfgArrays& a, uint32_t c) {
    const TabHdr* h = v.h;
    const uint32_t T = h->T, Z = h->Z, R = h->R, tid = threadIdx.x;
    if (tid < 32) {                    // the first warp sets the configuration up, one segment per lane
        Config k;
        uint32_t valid = 0;
        if (tid == 0) {
            k = config_of(pp.sp, c);
            cs.cfg = k;
            const uint32_t tp0 = h->tp_values[k.tpi];
            const uint64_t dm = (uint64_t)k.D * h->mbs_values[k.mi];
            valid = (k.D >= 1 && h->gbs % dm == 0 && h->heads % tp0 == 0) ? 1u : 0u;
            cs.valid = valid;
            cs.n_b = k.D >= 1 ? h->gbs / dm : 0;
            cs.ar_steps = (double)(2 * (uint64_t)(k.D > 0 ? k.D - 1 : 0));     // ring all-reduce: 2(D-1) messages
            cs.ar_coef = k.D > 0 ? cs.ar_steps / (double)k.D : 0.0;
            cs.n_items = ipow64(R, k.nseg - 1);
            cs.flat_base = pp.cfg_flat_base[c];
            cs._pad_head = 0;
            cs.packed = 0;             // decided at the end of the build, and only for valid configurations
            cs.cur_config = c;
            uint32_t n_lower = 0;
            if (pp.min_tp_only)
                for (uint32_t j = 0; j < pp.sp.n_tp; ++j) {
                    const uint32_t tj = pp.sp.tp_idx[j], tv = h->tp_values[tj];
                    if (tv < tp0 && h->heads % tv == 0 && n_lower < SAILOR_TP_MAX - 1) cs.lower_tpi[n_lower++] = tj;
                }
            cs.n_lower = n_lower;
        }
        const uint32_t P = __shfl_sync(FULL, k.P, 0), nseg = __shfl_sync(FULL, k.nseg, 0);
        const uint32_t D = __shfl_sync(FULL, k.D, 0), tp = h->tp_values[__shfl_sync(FULL, k.tpi, 0)];
        if (tid <= nseg) cs.seg_a[tid] = (tid * P + nseg - 1) / nseg;
        if (tid < nseg) {              // stages [lo, hi) of segment `tid`, counted per run in closed form
            const uint32_t lo = (tid * P + nseg - 1) / nseg, end = ((tid + 1) * P + nseg - 1) / nseg;
            const uint32_t extra = h->n_blocks % P;
            cs.need[tid] = D * tp * (end - lo);
            cs.oom_mask[tid] = 0;
            for (uint32_t j = 0; j < SAILOR_TP_MAX; ++j) cs.lower_fit[j][tid] = 0;
            uint32_t hi = (tid + 1 < nseg) ? end - 1 : end;      // a non-final segment's last stage is kept apart
            const uint32_t c3 = (hi == P && hi > lo) ? 1u : 0u;   // the final stage
            hi -= c3;
            const uint32_t c0 = (lo == 0 && h->has_embed && hi > lo) ? 1u : 0u;
            const uint32_t lo1 = lo + c0;
            const uint32_t top = hi < extra ? hi : extra;
            const uint32_t c1 = top > lo1 ? top - lo1 : 0u;
            cs.n_run[tid][0] = c0;
            cs.n_run[tid][1] = c1;
            cs.n_run[tid][2] = hi > lo1 ? (hi - lo1) - c1 : 0u;
            cs.n_run[tid][3] = c3;
        }
        uint32_t inv_lo = 0, inv_hi = 0;                          // digits whose type cannot host tp
        {
            const uint32_t d0 = tid, d1 = tid + 32;
            inv_lo = __ballot_sync(FULL, d0 < R && tp > h->gpn[d0 % T]);
            inv_hi = __ballot_sync(FULL, d1 < R && tp > h->gpn[d1 % T]);
        }
        if (tid == 0) cs.invalid_mask = ((uint64_t)inv_hi << 32) | inv_lo;
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
        if (sm.mem + h->reserved[g] > h->capacity[g]) atomicOr(&cs.oom_stage[i], 1ull << g);
        if (g == 0) cs.params[i] = sm.params;
    }
    for (uint32_t x = tid; x < cs.n_lower * P * T; x += PLAN_THREADS) {      // the same stages at the smaller degrees
        const uint32_t j = x / (P * T), i = (x / T) % P, g = x % T;
        const uint32_t nb = base + (i < extra ? 1u : 0u);
        const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
        const uint64_t inflight = (uint64_t)(P - i) < cs.n_b ? (uint64_t)(P - i) : cs.n_b;
        const StageMem sm = stage_memory(v, cs.lower_tpi[j], k.mi, k.rc, nb, e, hd, inflight);
        if (sm.mem + h->reserved[g] > h->capacity[g]) atomicOr(&cs.oom_stage[i], 1ull << (8 * (j + 1) + g));
    }
    for (uint32_t d = tid; d < R; d += PLAN_THREADS) {
        a.availv[d] = pp.avail[d];
        a.tz[d] = (d % T) | ((d / T) << 8);
    }
    __syncthreads();

    // phase B: boundary tables and per-(segment, digit) records
    const double msg = (double)v.p2p[k.mi];
    const uint64_t xbytes = 2 * cs.n_b * (uint64_t)k.D * v.p2p[k.mi];
    for (uint32_t x = tid; x < R * R; x += PLAN_THREADS) {
        const uint32_t dn = x / R, d = x % R;      // [next][this]
        a.c2x[x] = mul_rn(2.0, boundary_time(v, d % T, d / T, tp, dn % T, dn / T, tp, k.D, msg));
    }
    for (uint32_t x = tid; x < R * Z; x += PLAN_THREADS) {
        const uint32_t dn = x / Z, z = x % Z, zn = dn / T;      // [next digit][this zone]
        a.commx[x] = (z != zn) ? mul_rn((double)xbytes, v.egress[z * Z + zn]) : 0.0;
    }
    for (uint32_t x = tid; x < k.nseg * T; x += PLAN_THREADS) {
        const uint32_t s = x / T, g = x % T;
        a.fb_last[x] = a.fb[(cs.seg_a[s + 1] - 1) * T + g];
    }
    for (uint32_t x = tid; x < k.nseg * R; x += PLAN_THREADS) {
        const uint32_t s = x / R, d = x % R, g = d % T, z = d / T;
        const uint32_t sa = cs.seg_a[s], se = cs.seg_a[s + 1];
        // the last stage of a non-final segment talks to the next segment: its t is not in the runs
        const uint32_t t_end = (s + 1 < k.nseg) ? se - 1 : se;
        const double c2self = mul_rn(2.0, boundary_time(v, g, z, tp, g, z, tp, k.D, msg));
        SegRec r;
        for (int q = 0; q < N_RUNS; ++q) r.v[q] = 0.0;
        double tm = 0.0, sy = 0.0, up = 0.0;
        bool oom = false;
        unsigned long long oom_bits = 0;
        for (uint32_t i = sa; i < se; ++i) {
            oom_bits |= cs.oom_stage[i];
            if (i < t_end) {
                const double fbi = a.fb[i * T + g];
                const double t = (i + 1 < P) ? add_rn(fbi, c2self) : fbi;
                r.v[run_of(h, P, extra, i)] = t;
                tm = dmax(tm, t);
            }
            if (k.D > 1) sy = dmax(sy, allreduce_time(v, g, d, tp, k.D, cs.params[i], cs.ar_steps, cs.ar_coef));
            up = dmax(up, a.uu[i * T + g]);
            oom |= (cs.oom_stage[i] >> g) & 1u;
        }
        r.tmax = tm;
        r.sync = sy;
        r.upd = up;
        r.rate = mul_rn((double)(k.D * tp), v.price_s[d]);
        a.rec[x] = r;
        if (oom) atomicOr(reinterpret_cast<unsigned long long*>(&cs.oom_mask[s]), 1ull << d);
        for (uint32_t j = 0; j < cs.n_lower; ++j)
            if (!((oom_bits >> (8 * (j + 1) + g)) & 1ull))
                atomicOr(reinterpret_cast<unsigned long long*>(&cs.lower_fit[j][s]), 1ull << d);
    }
    __syncthreads();                   // the memory masks are complete
    if (tid < 32) {
        const uint32_t last = k.nseg - 1;
        const uint32_t need_last = cs.need[last];
        const uint32_t a_lo = __ballot_sync(FULL, tid < R && need_last <= a.availv[tid < R ? tid : 0]);
        const uint32_t a_hi = __ballot_sync(FULL, tid + 32 < R && need_last <= a.availv[tid + 32 < R ? tid + 32 : 0]);
        if (tid == 0) cs.avail_last = ((uint64_t)a_hi << 32) | a_lo;
        if (pp.live_mode) {
            // usable digits per segment (valid type, fits in memory): only prefixes made of them are
            // enumerated; lane d places digit d (and d + 32) at its rank among the set bits
            const uint64_t full = R == 64 ? ~0ull : ((1ull << R) - 1);
            uint64_t live = 1;
            for (uint32_t sgm = 0; sgm < k.nseg; ++sgm) {
                const uint64_t good = full & ~cs.invalid_mask & ~cs.oom_mask[sgm];
                const uint32_t g_lo = (uint32_t)good, g_hi = (uint32_t)(good >> 32);
                const uint32_t below = (1u << tid) - 1u;
                if ((g_lo >> tid) & 1u) cs.good_list[sgm][__popc(g_lo & below)] = (uint8_t)tid;
                if ((g_hi >> tid) & 1u) cs.good_list[sgm][__popc(g_lo) + __popc(g_hi & below)] = (uint8_t)(tid + 32);
                const uint32_t n = __popcll(good);
                if (tid == 0) {
                    cs.g_cnt[sgm] = n;
                    cs.g_magic[sgm] = n > 1 ? (uint32_t)(0x100000000ull / n) + 1u : 0u;
                }
                if (sgm + 1 < k.nseg) live *= n;
            }
            if (tid == 0) cs.live_items = live;
        }
        if (tid == 0) cs.packed = pp.live_mode;
    }
    __syncthreads();
}

// The tables of configuration `c` from the cache instead of building them: two straight copies, then the
// availability mask of the last segment, which is the only part that follows the snapshot.  Called by the
// whole block (after a barrier); ends synchronised.  `a.availv` holds the snapshot already.
__device__ void load_config(const PlanParams& pp, CfgShared& cs, CfgArrays& a, uint32_t R, uint32_t c) {
    const uint32_t tid = threadIdx.x;
    const uint4* src = pp.cfg_cache + (size_t)c * (pp.cache_head16 + pp.cache_arr16);
    for (uint32_t x = tid; x < pp.cache_head16; x += PLAN_THREADS) reinterpret_cast<uint4*>(&cs)[x] = src[x];
    for (uint32_t x = tid; x < pp.cache_arr16; x += PLAN_THREADS) reinterpret_cast<uint4*>(a.rec)[x] = src[pp.cache_head16 + x];
    __syncthreads();
    if (tid < 32) {
        const uint32_t need_last = cs.need[cs.cfg.nseg - 1];
        const uint32_t a_lo = __ballot_sync(FULL, tid < R && need_last <= a.availv[tid < R ? tid : 0]);
        const uint32_t a_hi = __ballot_sync(FULL, tid + 32 < R && need_last <= a.availv[tid + 32 < R ? tid + 32 : 0]);
        if (tid == 0) {
            cs.avail_last = ((uint64_t)a_hi << 32) | a_lo;
            cs.packed = cs.valid ? pp.live_mode : 0u;
            cs.cur_config = c;
        }
    }
    __syncthreads();
}

__device__ __forceinline__ uint64_t warp_or64(uint64_t x) {
    const uint32_t lo = __reduce_or_sync(FULL, (uint32_t)x);
    const uint32_t hi = __reduce_or_sync(FULL, (uint32_t)(x >> 32));
    return ((uint64_t)hi << 32) | lo;
}

struct Counters {
    uint32_t invalid, oom, over_avail, over_constr, feasible, total, pruned;
    double min_cost;
    double cfg_best;     // best feasible score seen in the current configuration
};

// Hand the block's best feasible score of configuration `c` to the per-configuration table (positive
// doubles order like their bit patterns) and start over.
__device__ __forceinline__ void flush_cfg_best(const PlanParams& pp, Counters& cnt, uint32_t c, uint32_t lane) {
    unsigned long long b = (unsigned long long)__double_as_longlong(cnt.cfg_best);
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(FULL, b, o);
        b = other < b ? other : b;
    }
    if (lane == 0 && b < (unsigned long long)__double_as_longlong(make_inf())) atomicMin(&pp.cfg_best[c], b);
    cnt.cfg_best = make_inf();
}

// Add a warp's per-thread counters to the block's 64-bit sums and clear them.
__device__ __forceinline__ void flush_counters(CfgShared& cs, Counters& cnt, uint32_t lane) {
    uint32_t* vals[7] = {&cnt.total, &cnt.invalid, &cnt.oom, &cnt.over_avail, &cnt.over_constr, &cnt.feasible,
                         &cnt.pruned};
#pragma unroll
    for (int j = 0; j < 7; ++j) {
        unsigned long long s = *vals[j];
#pragma unroll
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
        if (lane == 0 && s) atomicAdd(&cs.stat[j], s);
        *vals[j] = 0;
    }
}

// acc + v + v + ... (n times), one rounding per addition: the stage-by-stage sum of a run.
__device__ __forceinline__ double add_n(double acc, double v, uint32_t n) {
#pragma unroll 4
    for (uint32_t j = 0; j < n; ++j) acc = add_rn(acc, v);
    return acc;
}

// What a lane carries from its prefix into the walk over the last segment's digit.
struct ItemState {
    double acc, mx, sy, up, rate, cc;    // running sum / maxima / price rate / transfer cost of the prefix
    double fb_b;                         // f+b of the prefix's last stage (its message goes to the last digit)
    uint64_t ok, walk;                   // per last digit: feasible for this lane / worth visiting for the warp
    const SegRec* recs;                  // records of the last segment
    const double* c2x_col;               // c2x[.][d_prev]
    const double* comm_col;              // commx[.][z_prev]
};

// Time and cost of the W candidates that extend item `it` with last digits d .. d+W-1, evaluated
// side by side (W independent dependency chains; the stage loops run once for all of them).
template <int NSEG, int N2, int W>
__device__ __forceinline__ void eval_candidates(const CfgShared& cs, const ItemState& it, uint32_t Z, uint32_t R,
                                                uint32_t d, double nb, double (&t_iter)[W], double (&cost)[W]) {
    constexpr uint32_t last = NSEG - 1;
    const SegRec* rc = it.recs + d;
    double t_sum[W], t_max[W], c_comm[W], r[W];
#pragma unroll
    for (int w = 0; w < W; ++w) {
        t_sum[w] = it.acc; t_max[w] = it.mx; c_comm[w] = it.cc; r[w] = it.rate;
        if (NSEG > 1) {                                   // last stage of the prefix sends to digit d + w
            const double tb = add_rn(it.fb_b, it.c2x_col[(d + w) * R]);
            t_sum[w] = add_rn(t_sum[w], tb);
            t_max[w] = dmax(t_max[w], tb);
            c_comm[w] = add_rn(c_comm[w], it.comm_col[(d + w) * Z]);
        }
    }
    // the segment's stages in order: [stage 0] [stages with an extra block] [plain stages] [final stage];
    // the price-rate sum takes one term per stage alongside
#define SAILOR_STAGE(RUN)                                                          \
    _Pragma("unroll") for (int w = 0; w < W; ++w) {                                \
        t_sum[w] = add_rn(t_sum[w], rc[w].v[RUN]);                                 \
        r[w] = add_rn(r[w], rc[w].rate);                                           \
    }
    if (N2 >= 0) {
#pragma unroll
        for (int j = 0; j < N2; ++j) { SAILOR_STAGE(2) }
        SAILOR_STAGE(3)
    } else {
        const uint32_t n0 = cs.n_run[last][0], n1 = cs.n_run[last][1], n2 = cs.n_run[last][2], n3 = cs.n_run[last][3];
        if (n0) { SAILOR_STAGE(0) }
        for (uint32_t j = 0; j < n1; ++j) { SAILOR_STAGE(1) }
        uint32_t j = n2;
        for (; j >= 4; j -= 4) { SAILOR_STAGE(2) SAILOR_STAGE(2) SAILOR_STAGE(2) SAILOR_STAGE(2) }
        if (j & 2) { SAILOR_STAGE(2) SAILOR_STAGE(2) }
        if (j & 1) { SAILOR_STAGE(2) }
        if (n3) { SAILOR_STAGE(3) }
    }
#undef SAILOR_STAGE
#pragma unroll
    for (int w = 0; w < W; ++w) {
        t_max[w] = dmax(t_max[w], rc[w].tmax);
        const double t_pp = add_rn(t_sum[w], mul_rn(nb, t_max[w]));
        t_iter[w] = add_rn(add_rn(t_pp, dmax(it.sy, rc[w].sync)), dmax(it.up, rc[w].upd));
        cost[w] = add_rn(mul_rn(r[w], t_iter[w]), c_comm[w]);
    }
}

// ---- the binary32 screen: the same walk from the rounded tables ---------------------------------------------
__device__ __forceinline__ float fadd(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ float fmul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ float fmaxf_sel(float a, float b) { return fmaxf(a, b); }      // one instruction in binary32; no NaN occurs

struct ItemState32 {
    float acc, mx, sy, up, rate, cc, fb_b;
    const SegRec32* recs;
    const float* c2x_col;
    const float* comm_col;
};

template <int NSEG, int N2, int W>
__device__ __forceinline__ void eval_candidates32(const CfgShared& cs, const ItemState32& it, uint32_t Z, uint32_t R,
                                                  uint32_t d, float nb, float (&t_iter)[W], float (&cost)[W]) {
    constexpr uint32_t last = NSEG - 1;
    const SegRec32* rc = it.recs + d;
    float t_sum[W], t_max[W], c_comm[W], r[W];
#pragma unroll
    for (int w = 0; w < W; ++w) {
        t_sum[w] = it.acc; t_max[w] = it.mx; c_comm[w] = it.cc; r[w] = it.rate;
        if (NSEG > 1) {
            const float tb = fadd(it.fb_b, it.c2x_col[(d + w) * R]);
            t_sum[w] = fadd(t_sum[w], tb);
            t_max[w] = fmaxf_sel(t_max[w], tb);
            c_comm[w] = fadd(c_comm[w], it.comm_col[(d + w) * Z]);
        }
    }
#define SAILOR_STAGE32(RUN)                                                        \
    _Pragma("unroll") for (int w = 0; w < W; ++w) {                                \
        t_sum[w] = fadd(t_sum[w], rc[w].v[RUN]);                                   \
        r[w] = fadd(r[w], rc[w].rate);                                             \
    }
    if (N2 >= 0) {
#pragma unroll
        for (int j = 0; j < N2; ++j) { SAILOR_STAGE32(2) }
        SAILOR_STAGE32(3)
    } else {
        const uint32_t n0 = cs.n_run[last][0], n1 = cs.n_run[last][1], n2 = cs.n_run[last][2], n3 = cs.n_run[last][3];
        if (n0) { SAILOR_STAGE32(0) }
        for (uint32_t j = 0; j < n1; ++j) { SAILOR_STAGE32(1) }
        uint32_t j = n2;
        for (; j >= 4; j -= 4) { SAILOR_STAGE32(2) SAILOR_STAGE32(2) SAILOR_STAGE32(2) SAILOR_STAGE32(2) }
        if (j & 2) { SAILOR_STAGE32(2) SAILOR_STAGE32(2) }
        if (j & 1) { SAILOR_STAGE32(2) }
        if (n3) { SAILOR_STAGE32(3) }
    }
#undef SAILOR_STAGE32
#pragma unroll
    for (int w = 0; w < W; ++w) {
        t_max[w] = fmaxf_sel(t_max[w], rc[w].tmax);
        const float t_pp = fadd(t_sum[w], fmul(nb, t_max[w]));
        t_iter[w] = fadd(fadd(t_pp, fmaxf_sel(it.sy, rc[w].sync)), fmaxf_sel(it.up, rc[w].upd));
        cost[w] = fadd(fmul(r[w], t_iter[w]), c_comm[w]);
    }
}

// Binary32 pass over the candidates of one item: the lane's best score and cheapest cost, both approximate.
template <int NSEG, int OBJ, int N2>
__device__ __forceinline__ void walk_fast32(const CfgShared& cs, const ItemState32& it, uint64_t ok, uint64_t walk,
                                            uint32_t Z, uint32_t R, float& best, float& min_cost) {
    const float nb = (float)cs.n_b;
    constexpr uint32_t U = PLAN_DIGITS_PER_STEP;
    for (uint32_t half = 0; half * 32 < R; ++half) {
        const uint32_t wm = (uint32_t)(walk >> (32 * half)), om = (uint32_t)(ok >> (32 * half));
        const uint32_t d_end = min(R - 32 * half, 32u);
        for (uint32_t dd = 0; dd < d_end; dd += U) {
            if (!((wm >> dd) & ((1u << U) - 1u))) continue;   // warp-uniform
            float t[U], c[U];
            eval_candidates32<NSEG, N2, (int)U>(cs, it, Z, R, 32 * half + dd, nb, t, c);
#pragma unroll
            for (uint32_t u = 0; u < U; ++u) {
                const bool g = (om >> (dd + u)) & 1u;
                const float sc = OBJ == SAILOR_OBJ_MAX_THROUGHPUT ? t[u] : OBJ == SAILOR_OBJ_MIN_COST ? c[u] : fmul(t[u], c[u]);
                min_cost = fminf(min_cost, g ? c[u] : min_cost);
                best = fminf(best, g ? sc : best);
            }
        }
    }
}

template <int OBJ>
__device__ __forceinline__ double score_of(double t_iter, double cost) {
    return OBJ == SAILOR_OBJ_MAX_THROUGHPUT ? t_iter : OBJ == SAILOR_OBJ_MIN_COST ? cost : mul_rn(t_iter, cost);
}

template <bool CONSTR>
__device__ __forceinline__ bool within(const PlanParams& pp, double budget, double t_iter, double cost) {
    bool good = true;
    if (CONSTR) {
        if (budget > 0.0) good &= !(cost > budget);
        if (pp.min_rate > 0.0) good &= !(1.0 / t_iter < pp.min_rate);
    }
    return good;
}

// Fast pass over the candidates of one item, several digits per step (independent dependency
// chains per thread): tracks the lane's best score, the feasible count and the cheapest cost.
// No votes, no list updates.  Tables are padded, so a step may read (and mask out) digits >= R.
template <int NSEG, int OBJ, bool CONSTR, int N2>
__device__ __forceinline__ void walk_fast(const PlanParams& pp, const CfgShared& cs, const ItemState& it,
                                          uint32_t Z, uint32_t R, double budget, double& best, uint32_t& feas,
                                          double& min_cost) {
    const double nb = (double)cs.n_b;
    constexpr uint32_t U = PLAN_DIGITS_PER_STEP;
    for (uint32_t half = 0; half * 32 < R; ++half) {
        const uint32_t wm = (uint32_t)(it.walk >> (32 * half)), om = (uint32_t)(it.ok >> (32 * half));
        const uint32_t d_end = min(R - 32 * half, 32u);
        for (uint32_t dd = 0; dd < d_end; dd += U) {
            if (!((wm >> dd) & ((1u << U) - 1u))) continue;   // warp-uniform
            const uint32_t d = 32 * half + dd;
            double t[U], c[U];
            eval_candidates<NSEG, N2, (int)U>(cs, it, Z, R, d, nb, t, c);
#pragma unroll
            for (uint32_t u = 0; u < U; ++u) {
                const bool g = ((om >> (dd + u)) & 1u) && within<CONSTR>(pp, budget, t[u], c[u]);
                const double sc = score_of<OBJ>(t[u], c[u]);
                if (CONSTR) feas += (uint32_t)g;
                min_cost = (g && c[u] < min_cost) ? c[u] : min_cost;
                best = (g && sc < best) ? sc : best;
            }
        }
    }
}

// Rare second pass over an item: the same arithmetic, one digit at a time, and every candidate that
// may enter the warp's top-k list is offered to it (warp-synchronous).  Nothing is counted.
template <int NSEG, int OBJ, bool CONSTR, int N2>
__device__ __forceinline__ void walk_offer(const PlanParams& pp, const CfgShared& cs, const ItemState& it,
                                           uint32_t Z, uint32_t R, double budget, uint64_t item_flat,
                                           WarpTopK& top, uint32_t lane, double outer_thr, double& min_cost) {
    const double nb = (double)cs.n_b;
    for (uint32_t d = 0; d < R; ++d) {
        if (!((it.walk >> d) & 1ull)) continue;               // warp-uniform
        double t1[1], c1[1];
        eval_candidates<NSEG, N2, 1>(cs, it, Z, R, d, nb, t1, c1);
        const double t = t1[0], c = c1[0];
        const bool good = ((it.ok >> d) & 1ull) && within<CONSTR>(pp, budget, t, c);
        const double score = score_of<OBJ>(t, c);
        min_cost = (good && c < min_cost) ? c : min_cost;      // (the fast pass of the exact search has seen it already)
        const bool want = good && score <= top.thr_score && score <= outer_thr;
        if (__any_sync(FULL, want)) top.offer(want, score, item_flat + d, pp.k, lane);
    }
}

// One item per lane: fixed prefix digits, walk the last segment's digit.
// N2 >= 0 fixes the shape of the last segment at compile time (N2 plain stages, then the final
// stage, nothing else), which makes the candidate loop straight-line code; N2 < 0 is the general form.
template <int NSEG, int OBJ, bool CONSTR, int N2, bool SCREEN>
__device__ __forceinline__ void run_items(const PlanParams& pp, const CfgShared& cs, const CfgArrays& a,
                                          uint32_t T, uint32_t Z, uint32_t R, uint32_t q, bool active,
                                          uint64_t item_flat, double budget, WarpTopK& top, Counters& cnt,
                                          uint32_t lane) {
    constexpr uint32_t last = NSEG - 1;
    // ---- prefix: segments 0 .. NSEG-2 --------------------------------------------------------
    uint32_t dg[NSEG > 1 ? NSEG - 1 : 1];
    {
        uint32_t x = active ? q : 0;
        if (cs.packed) {                                   // mixed radix over the usable digits of each segment
#pragma unroll
            for (int s = NSEG - 2; s >= 0; --s) {
                const uint32_t n = cs.g_cnt[s];
                const uint32_t y = n > 1 ? __umulhi(x, cs.g_magic[s]) : x;   // x / n
                dg[s] = active ? cs.good_list[s][x - y * n] : 0u;
                x = y;
            }
        } else {
#pragma unroll
            for (int s = NSEG - 2; s >= 0; --s) {
                const uint32_t y = R == 1 ? x : __umulhi(x, cs.magic);     // x / R
                dg[s] = x - y * R;
                x = y;
            }
        }
    }
    if (cs.packed) {                                       // the item's flat index follows from its digits
        uint64_t pf = 0;
#pragma unroll
        for (int s = 0; s < NSEG - 1; ++s) pf = pf * R + dg[s];
        item_flat = cs.flat_base + pf * R;
    }
    // ---- status of the prefix: node validity, memory, availability (integer work only) ------------
    bool p_inv = false, p_oom = false, p_over = false;
#pragma unroll
    for (int s = 0; s < NSEG - 1; ++s) {
        const uint32_t d = dg[s];
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
    const uint64_t fit_l = valid_l & ~cs.oom_mask[last];
    uint64_t drop = 0;            // last digits at which the whole plan also fits with a smaller degree
    if (pp.min_tp_only)
        for (uint32_t j = 0; j < cs.n_lower; ++j) {
            bool pf = true;
#pragma unroll
            for (int s = 0; s < NSEG - 1; ++s) pf &= (cs.lower_fit[j][s] >> dg[s]) & 1;
            if (pf) drop |= cs.lower_fit[j][last];
        }
    const uint64_t good_l = fit_l & ~drop;
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
    if (cs.packed) {                                      // total, invalid and oom were added in closed form
        cnt.pruned += __popcll(fit_l) - __popcll(good_l);
        if (p_over) { cnt.over_avail += __popcll(good_l); ok = 0; }
        else cnt.over_avail += __popcll(good_l) - __popcll(ok);
    } else if (p_inv) { cnt.total += n_range; cnt.invalid += n_range; ok = 0; }
    else {
        cnt.total += n_range;
        cnt.invalid += n_range - __popcll(valid_l);
        if (p_oom) { cnt.oom += __popcll(valid_l); ok = 0; }
        else {
            cnt.oom += __popcll(valid_l) - __popcll(fit_l);
            cnt.pruned += __popcll(fit_l) - __popcll(good_l);
            if (p_over) { cnt.over_avail += __popcll(good_l); ok = 0; }
            else cnt.over_avail += __popcll(good_l) - __popcll(ok);
        }
    }
    const uint32_t n_ok = __popcll(ok);
    if (!CONSTR) cnt.feasible += n_ok;

    // ---- the candidates -----------------------------------------------------------------------
    const uint64_t walk = pp.eval_all ? warp_or64(range) : warp_or64(ok);   // warp-uniform: skip dead digits
    if (walk == 0) {                                      // nothing to evaluate for any lane of the warp
        return;
    }
    // ---- running sums of the prefix, in stage order ---------------------------------------------
    double acc = 0.0, mx = 0.0, sy = 0.0, up = 0.0, rate = 0.0, cc = 0.0;
#pragma unroll
    for (int s = 0; s < NSEG - 1; ++s) {
        const uint32_t d = dg[s];
        const SegRec& rc = a.rec[s * R + d];
#pragma unroll
        for (int r = 0; r < N_RUNS - 1; ++r) acc = add_n(acc, rc.v[r], cs.n_run[s][r]);   // run 3 is the final stage
        mx = dmax(mx, rc.tmax);
        sy = dmax(sy, rc.sync);
        up = dmax(up, rc.upd);
        rate = add_n(rate, rc.rate, cs.seg_a[s + 1] - cs.seg_a[s]);
        if (s < NSEG - 2) {                               // the segment's last stage sends to the next prefix digit
            const uint32_t dn = dg[s + 1];
            const double tb = add_rn(a.fb_last[s * T + (a.tz[d] & 0xff)], a.c2x[dn * R + d]);
            acc = add_rn(acc, tb);
            mx = dmax(mx, tb);
            cc = add_rn(cc, a.commx[dn * Z + (a.tz[d] >> 8)]);
        }
    }
    ItemState it;
    it.acc = acc; it.mx = mx; it.sy = sy; it.up = up; it.rate = rate; it.cc = cc;
    it.ok = ok;
    it.walk = walk;
    it.fb_b = 0.0;
    uint32_t d_prev = 0, z_prev = 0;
    if (NSEG > 1) {
        d_prev = dg[NSEG > 1 ? NSEG - 2 : 0];
        z_prev = a.tz[d_prev] >> 8;
        it.fb_b = a.fb_last[(NSEG > 1 ? NSEG - 2 : 0) * T + (a.tz[d_prev] & 0xff)];
    }
    it.recs = a.rec + last * R;
    it.c2x_col = a.c2x + d_prev;
    it.comm_col = a.commx + z_prev;

    if (SCREEN) {
        // binary32 first; the item is walked exactly only if it may hold a member of the top-k or the cheapest plan
        ItemState32 s32;
        s32.acc = __double2float_rn(acc); s32.mx = __double2float_rn(mx); s32.sy = __double2float_rn(sy);
        s32.up = __double2float_rn(up); s32.rate = __double2float_rn(rate); s32.cc = __double2float_rn(cc);
        s32.fb_b = __double2float_rn(it.fb_b);
        s32.recs = a.rec32 + last * R;
        s32.c2x_col = a.c2x32 + d_prev;
        s32.comm_col = a.commx32 + z_prev;
        const float f_inf = __int_as_float(0x7f800000);
        float best32 = f_inf, minc32 = f_inf;
        walk_fast32<NSEG, OBJ, N2>(cs, s32, ok, walk, Z, R, best32, minc32);
        const double outer_thr = __longlong_as_double((long long)*reinterpret_cast<const volatile unsigned long long*>(&cs.thr_bits));
        const double outer_minc = __longlong_as_double((long long)*reinterpret_cast<const volatile unsigned long long*>(&cs.minc_bits));
        const double thr = top.thr_score < outer_thr ? top.thr_score : outer_thr;
        const bool need = best32 < f_inf && ((double)best32 <= thr * (1.0 + SCREEN_BAND) || (double)minc32 <= outer_minc * (1.0 + SCREEN_BAND));
        if (__any_sync(FULL, need)) {
            const double before = top.thr_score, mc_before = cnt.min_cost;
            walk_offer<NSEG, OBJ, CONSTR, N2>(pp, cs, it, Z, R, budget, item_flat, top, lane, outer_thr, cnt.min_cost);
            if (lane == 0 && top.thr_score < before)
                atomicMin(const_cast<unsigned long long*>(&cs.thr_bits), (unsigned long long)__double_as_longlong(top.thr_score));
            if (cnt.min_cost < mc_before)
                atomicMin(const_cast<unsigned long long*>(&cs.minc_bits), (unsigned long long)__double_as_longlong(cnt.min_cost));
        }
        return;
    }
    // fast pass: no votes, no list updates; each lane keeps its item's best score
    double best = make_inf();
    uint32_t feas = 0;
    walk_fast<NSEG, OBJ, CONSTR, N2>(pp, cs, it, Z, R, budget, best, feas, cnt.min_cost);
    cnt.cfg_best = best < cnt.cfg_best ? best : cnt.cfg_best;
    if (CONSTR) {
        cnt.feasible += feas;
        cnt.over_constr += n_ok - feas;
    }
    // rare: some lane's item holds a candidate that may enter the warp's list; walk again and offer
    // (a candidate worse than the k-th best of ANY warp's list cannot be among the k best overall: the block keeps
    // the lowest such score its warps and the other blocks have reached; equal scores still pass, the list decides)
    const double outer_thr = __longlong_as_double((long long)*reinterpret_cast<const volatile unsigned long long*>(&cs.thr_bits));
    if (!pp.cost_only && __any_sync(FULL, best < make_inf() && best <= top.thr_score && best <= outer_thr)) {   // best == inf: no feasible candidate
        const double before = top.thr_score;
        walk_offer<NSEG, OBJ, CONSTR, N2>(pp, cs, it, Z, R, budget, item_flat, top, lane, outer_thr, cnt.min_cost);
        if (lane == 0 && top.thr_score < before)
            atomicMin(const_cast<unsigned long long*>(&cs.thr_bits), (unsigned long long)__double_as_longlong(top.thr_score));
    }
}

// End of a pass, run by the one block that hands in its list last (no block waits for another: every block
// adds one to Ctrl::blocks_done after its list is written, and the block that reads gridDim.x - 1 knows all the
// lists are in memory).  Merges the blocks' lists, simulates the winners in full for the result records, copies
// the counters next to them, hands `factor x best cost` to a following pass, and puts the counters back to
// their starting values.  `v` is the block's own view of the static tables (already in shared memory); `s_hits`
// (PLAN_WARPS lists) and `s_cnt` (R x SAILOR_K_MAX words) are scratch in shared memory.
__device__ __noinline__ void finish_pass(const PlanParams& pp, const TabView& v, Hit (*s_hits)[SAILOR_K_MAX],
                                         uint32_t* s_cnt, uint32_t* s_n, uint32_t n_partial) {
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = PLAN_WARPS;
    if (pp.cost_only) {
        // the cheapest-plan pass of a budget-factor search: all the next pass needs is factor x the cheapest feasible
        // cost, which every block has already folded into Ctrl::min_cost_bits (the same bits a full simulation of
        // that plan gives: one operation order everywhere)
        if (tid == 0) {
            volatile Ctrl* live = pp.ctrl;
            const bool any = live->stats[5] != 0;
            const double cheapest = __longlong_as_double((long long)live->min_cost_bits);
            pp.ctrl->budget = any ? mul_rn(pp.next_budget_factor, cheapest) : make_inf();
            Ctrl* c = pp.ctrl;
            c->work_counter = 0;
            for (int q = 0; q < 7; ++q) c->stats[q] = 0;
            c->wave_chunks = 0;
            c->n_cfg_evaluated = 0;
            c->min_cost_bits = COST_BITS_START;
            c->thr_bits = COST_BITS_START;
            c->n_found = 0;
        }
        return;
    }
    // The k best of all lists lie in the k lists with the best first elements: k elements (those heads) are at
    // least as good as the k-th best head, and a list whose head is worse holds nothing better than its head.
    // So: the k best heads first (one element per list, all loads in flight together), then only those lists.
    // (Every block writes all k slots of its list, empty ones as (+inf, ~0); read them in L2, other SMs wrote them.)
    auto load_hit = [&](uint32_t b, uint32_t slot, double& sc, uint64_t& fl) {
        const double2 raw = __ldcg(reinterpret_cast<const double2*>(&pp.partial[(size_t)b * SAILOR_K_MAX + slot]));
        sc = raw.x;
        fl = (uint64_t)__double_as_longlong(raw.y);
    };
    WarpTopK top;
    top.init();
    const uint32_t rounds = (n_partial + PLAN_THREADS - 1) / PLAN_THREADS;
    for (uint32_t r = 0; r < rounds; ++r) {
        const uint32_t b = r * PLAN_THREADS + tid;
        double hs = make_inf();
        uint64_t hf = ~0ull;
        if (b < n_partial) load_hit(b, 0, hs, hf);
        top.offer(hf != ~0ull && (hs < top.thr_score || (hs == top.thr_score && hf < top.thr_flat)), hs, hf, pp.k, lane);
    }
    auto tree_merge = [&]() {          // the warps' lists into warp 0's, through shared memory
        s_hits[warp][lane].score = top.score;
        s_hits[warp][lane].flat = top.flat;
        __syncthreads();
        for (uint32_t step = 1; step < nw; step <<= 1) {
            if ((warp & (2 * step - 1)) == 0 && warp + step < nw) {
                top.merge_sorted(s_hits[warp + step][lane].score, s_hits[warp + step][lane].flat, pp.k, lane);
                s_hits[warp][lane].score = top.score;
                s_hits[warp][lane].flat = top.flat;
            }
            __syncthreads();
        }
    };
    tree_merge();
    const double cut_s = s_hits[0][pp.k - 1].score;          // the k-th best head (or (+inf, ~0): fewer than k lists hold anything)
    const uint64_t cut_f = s_hits[0][pp.k - 1].flat;
    uint32_t* sel = s_cnt;                                    // the chosen lists (at most k), then reused as counters
    if (tid == 0) *s_n = 0;
    __syncthreads();
    for (uint32_t r = 0; r < rounds; ++r) {
        const uint32_t b = r * PLAN_THREADS + tid;
        double hs = make_inf();
        uint64_t hf = ~0ull;
        if (b < n_partial) load_hit(b, 0, hs, hf);
        if (hf != ~0ull && (hs < cut_s || (hs == cut_s && hf <= cut_f))) sel[atomicAdd(s_n, 1u)] = b;
    }
    __syncthreads();
    const uint32_t n_sel = *s_n;
    top.init();
    for (uint32_t q = warp; q < n_sel; q += nw) {
        double ls = make_inf();
        uint64_t lf = ~0ull;
        if (lane < pp.k) load_hit(sel[q], lane, ls, lf);
        top.merge_sorted(ls, lf, pp.k, lane);
    }
    __syncthreads();                                           // `sel` has been read by everyone
    tree_merge();
    if (warp == 0) {
        const bool have = lane < pp.k && top.flat != ~0ull;
        const uint32_t n = __popc(__ballot_sync(FULL, have));
        if (lane == 0) *s_n = n;
    }
    __syncthreads();
    // the winners are simulated in full for the result records, all at once: winner j by lane j / PLAN_WARPS of warp
    // j % PLAN_WARPS (each is a long single-thread dependency chain of table look-ups; spread over the warps, at
    // most four different plans share a warp's instruction stream)
    const uint32_t n = *s_n;
    {
        const uint32_t j = lane * nw + warp;
        if (lane < (SAILOR_K_MAX + nw - 1) / nw && j < n) {
            sailor_result r;
            r.flat = s_hits[0][j].flat;
            r.score = s_hits[0][j].score;
            r._pad = 0;
            decode_flat(pp.sp, v.h->T, v.h->Z, r.flat, &r.plan);
            const SimOut o = simulate_record(v, pp.avail, r.plan, s_cnt + j, SAILOR_K_MAX);
            r.t_iter = o.t_iter;
            r.cost = o.cost;
            r.peak_mem = o.peak_mem;
            r.status = o.status;
            pp.out->results[j] = r;
            if (j == 0 && pp.next_budget_factor > 0.0) pp.ctrl->budget = mul_rn(pp.next_budget_factor, o.cost);
        }
    }
    if (tid == 0) {
        if (n == 0 && pp.next_budget_factor > 0.0) pp.ctrl->budget = make_inf();
        // the counters as they stand (every block's contribution is in: atomics, then its blocks_done increment)
        volatile Ctrl* live = pp.ctrl;
        Ctrl c;
        c.work_counter = live->work_counter;
        c.blocks_done = live->blocks_done;
        for (int q = 0; q < 7; ++q) c.stats[q] = live->stats[q];
        c.wave_chunks = live->wave_chunks;
        c.n_cfg_evaluated = live->n_cfg_evaluated;
        c.min_cost_bits = live->min_cost_bits;
        c.thr_bits = live->thr_bits;
        c.error = live->error;
        c.n_found = n;
        pp.out->ctrl = c;
    }
    __syncthreads();                   // the budget of the next pass is written (thread 0 or warp 0's lane 0)
    if (tid == 0) {
        pp.out->ctrl.budget = *reinterpret_cast<volatile double*>(&pp.ctrl->budget);
        Ctrl* live = pp.ctrl;          // back to the starting values; the budget stays for the next pass
        live->work_counter = 0;
        for (int q = 0; q < 7; ++q) live->stats[q] = 0;
        live->wave_chunks = 0;
        live->n_cfg_evaluated = 0;
        live->min_cost_bits = COST_BITS_START;
        live->thr_bits = COST_BITS_START;
        if (!(pp.next_budget_factor > 0.0)) live->error = 0;   // a following pass of the same call keeps the flag
        live->n_found = 0;
    }
}

// FUSED: the block that hands in its list last also ends the pass (one launch per pass: what small searches, bound
// by launch and hand-over latencies, want).  Not FUSED: the lists are left for finish_kernel (the call inside the
// kernel costs the candidate loop a few registers, which long searches would pay for in every iteration).
// SCREEN: candidates are evaluated in binary32 first (unconstrained searches; see SCREEN_BAND).
template <int OBJ, bool CONSTR, bool FUSED, bool SCREEN = false>
__global__ void __launch_bounds__(PLAN_THREADS, SCREEN ? PLAN_SCREEN_BLOCKS : PLAN_MIN_BLOCKS) plan_kernel(const __grid_constant__ PlanParams pp) {
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
    carve(dyn, static_bytes, pp.p_max, T, Z, a, pp.n_config, SCREEN);

    if (tid == 0) {
        cs.cur_config = 0xffffffffu;
        cs.minc_bits = COST_BITS_START;
        cs.magic = (uint32_t)(0x100000000ull / (gh->R ? gh->R : 1u)) + 1u;      // for x / R, see CfgShared
    }
    if (tid < 7) cs.stat[tid] = 0;
    if (tid == 7) cs.thr_bits = *reinterpret_cast<volatile unsigned long long*>(&pp.ctrl->thr_bits);
    // the padding digit of the tables is read (and masked out) by the two-digit steps: keep it finite
    for (uint32_t x = tid; x < PLAN_PAD * sizeof(SegRec) / 8; x += PLAN_THREADS)
        reinterpret_cast<double*>(a.rec + (size_t)SAILOR_SEG_MAX * R)[x] = 0.0;
    for (uint32_t x = tid; x < PLAN_PAD * R; x += PLAN_THREADS) a.c2x[(size_t)R * R + x] = 0.0;
    for (uint32_t x = tid; x < PLAN_PAD * Z; x += PLAN_THREADS) a.commx[(size_t)R * Z + x] = 0.0;
    for (uint32_t d = tid; d < R; d += PLAN_THREADS) {      // what does not depend on the configuration
        a.availv[d] = pp.avail[d];
        a.tz[d] = (d % T) | ((d / T) << 8);
    }
    // the chunk offsets are searched once per run of chunks and read once per chunk: keep a copy next to the tables
    // (the waves of a degree-order search rewrite them between launches, so every launch copies them afresh)
    const bool tab_local = pp.n_config < PLAN_CFG_SMEM;
    if (tab_local)
        for (uint32_t x = tid; x <= pp.n_config; x += PLAN_THREADS) a.chunk_tab[x] = pp.cfg_chunk_start[x];
    const uint32_t* chunk_start = tab_local ? a.chunk_tab : pp.cfg_chunk_start;
    WarpTopK top;
    top.init();
    if (pp.carry_lists && warp == 0) {     // a later wave of one search: go on from the list this block left behind
        if (lane < pp.partial_n[blockIdx.x]) {
            top.score = pp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].score;
            top.flat = pp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].flat;
        }
        top.thr_score = __shfl_sync(FULL, top.score, pp.k - 1);
        top.thr_flat = __shfl_sync(FULL, top.flat, pp.k - 1);
    }
    Counters cnt = {0, 0, 0, 0, 0, 0, 0, make_inf(), make_inf()};
    const double budget = pp.budget_from_ctrl ? pp.ctrl->budget : pp.budget;
    const uint32_t chunk_lo = pp.chunk_hi_dev ? 0u : pp.chunk_lo;
    const uint32_t chunk_hi = pp.chunk_hi_dev ? *pp.chunk_hi_dev : pp.chunk_hi;
    __syncthreads();

    uint32_t c = 0;     // configuration of the current chunk (monotone within a batch)
    bool first_round = true;
    for (;;) {
        if (tid == 0) {
            // every block starts with the chunk of its own number (no counter involved: small searches are bound by
            // such round trips); the rest is handed out by guided self-scheduling: long runs of consecutive chunks
            // first (a block then stays inside one configuration and changes its tables rarely), single chunks at
            // the end (even finish)
            const uint32_t n_chunks = chunk_hi - chunk_lo;
            if (!first_round) {      // trade thresholds with the other blocks
                const unsigned long long theirs = *reinterpret_cast<volatile unsigned long long*>(&pp.ctrl->thr_bits);
                const unsigned long long ours = *reinterpret_cast<volatile unsigned long long*>(&cs.thr_bits);
                if (ours < theirs) atomicMin(&pp.ctrl->thr_bits, ours);
                else if (theirs < ours) atomicMin(&cs.thr_bits, theirs);
            }
            if (first_round) {
                cs.next_chunk = chunk_lo + min(blockIdx.x, n_chunks);
                cs.batch_len = 1;
            } else if (n_chunks <= gridDim.x) {
                cs.next_chunk = chunk_hi;                    // every chunk had a block of its own
                cs.batch_len = 1;
            } else {
                const uint32_t rest = n_chunks - gridDim.x;
                const uint32_t seen = *reinterpret_cast<volatile unsigned int*>(&pp.ctrl->work_counter);
                const uint32_t left = seen < rest ? rest - seen : 0u;
                const uint32_t len = max(1u, left / (gridDim.x * 4u));
                const uint32_t got = atomicAdd(&pp.ctrl->work_counter, len);
                cs.next_chunk = got < rest ? chunk_lo + gridDim.x + got : chunk_hi;
                cs.batch_len = len;
            }
        }
        first_round = false;
        __syncthreads();
        const uint32_t first = cs.next_chunk;
        if (first >= chunk_hi) break;
        const uint32_t end = min(first + cs.batch_len, chunk_hi);
        {   // configuration of the first chunk: binary search (uniform)
            uint32_t lo = 0, hi = pp.n_config;
            while (hi - lo > 1) {
                const uint32_t mid = (lo + hi) >> 1;
                if (chunk_start[mid] <= first) lo = mid; else hi = mid;
            }
            c = lo;
        }
        for (uint32_t ch = first; ch < end; ++ch) {
            while (ch >= chunk_start[c + 1]) ++c;
            if (cs.cur_config != c) {
                if (pp.cfg_best && cs.cur_config != 0xffffffffu) flush_cfg_best(pp, cnt, cs.cur_config, lane);
                __syncthreads();
                if (pp.cfg_cache) load_config(pp, cs, a, R, c);
                else build_config(pp, v, cs, a, c);
                if (SCREEN) round_config32(a, R, Z);
            }
            const uint32_t q = (ch - chunk_start[c]) * PLAN_THREADS + tid;    // < R^3 + 256 <= 2^18 + 256
            const bool active = q < (cs.packed ? cs.live_items : cs.n_items);
            const uint64_t item_flat = cs.flat_base + (uint64_t)q * R;
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
            // the bulk of every space has four segments: pick the straight-line loop for its common shapes
            const int fixed = (cs.n_run[3][0] == 0 && cs.n_run[3][1] == 0 && cs.n_run[3][3] == 1 && cs.n_run[3][2] <= 3)
                                  ? (int)cs.n_run[3][2] : -1;
#define SAILOR_RUN(NS, NF) run_items<NS, OBJ, CONSTR, NF, SCREEN>(pp, cs, a, T, Z, R, q, active, item_flat, budget, top, cnt, lane)
            switch (cs.cfg.nseg) {
                case 1: SAILOR_RUN(1, -1); break;
                case 2: SAILOR_RUN(2, -1); break;
                case 3: SAILOR_RUN(3, -1); break;
                default:
                    switch (fixed) {
                        case 0: SAILOR_RUN(4, 0); break;
                        case 1: SAILOR_RUN(4, 1); break;
                        case 2: SAILOR_RUN(4, 2); break;
                        case 3: SAILOR_RUN(4, 3); break;
                        default: SAILOR_RUN(4, -1); break;
                    }
                    break;
            }
#undef SAILOR_RUN
        }
        // per-thread counters are 32 bits wide: hand them to the block's 64-bit sums in time
        if (__any_sync(FULL, cnt.total > (1u << 30))) flush_counters(cs, cnt, lane);
        __syncthreads();     // next_chunk and the tables are reused
    }

    // ---- block reduction: counters, then the warps' lists ---------------------------------------
    if (pp.cfg_best && cs.cur_config != 0xffffffffu) flush_cfg_best(pp, cnt, cs.cur_config, lane);
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
    if (tid < 7 && cs.stat[tid]) atomicAdd(&pp.ctrl->stats[tid], cs.stat[tid]);
    if (warp == 0) {
        for (uint32_t w = 1; w < PLAN_WARPS; ++w) {
            if (s_hits[w][0].flat == ~0ull) continue;    // an empty list
            top.merge_sorted(s_hits[w][lane].score, s_hits[w][lane].flat, pp.k, lane);
        }
        const uint32_t n = __popc(__ballot_sync(FULL, top.flat != ~0ull && lane < pp.k));
        if (lane < pp.k) {
            pp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].score = top.score;
            pp.partial[(size_t)blockIdx.x * SAILOR_K_MAX + lane].flat = top.flat;
        }
        if (lane == 0) pp.partial_n[blockIdx.x] = n;
    }
    if (FUSED) {
        // hand the list in; the block that does so last ends the launch (and, in a pass's final launch, the pass)
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned int before = atomicAdd(&pp.ctrl->blocks_done, 1u);
            cs.next_chunk = (before == gridDim.x - 1) ? 1u : 0u;
            if (before == gridDim.x - 1) {
                pp.ctrl->blocks_done = 0;                    // the next launch counts from zero
                if (!pp.finish) pp.ctrl->work_counter = 0;   // (a finishing launch resets all counters below)
            }
        }
        __syncthreads();
        if (cs.next_chunk && pp.finish) {
            __threadfence();
            finish_pass(pp, v, s_hits, reinterpret_cast<uint32_t*>(a.rec), &cs.batch_len, gridDim.x);
        }
    }
}

// The end of a pass as a launch of its own (one block), after a search kernel that is not FUSED.
__global__ void __launch_bounds__(PLAN_THREADS) finish_kernel(const __grid_constant__ PlanParams pp, uint32_t n_partial) {
    extern __shared__ __align__(16) unsigned char dyn[];      // the static tables, then R x SAILOR_K_MAX counters
    __shared__ Hit s_hits[PLAN_WARPS][SAILOR_K_MAX];
    __shared__ uint64_t mbar;
    __shared__ uint32_t s_n;
    const uint32_t tid = threadIdx.x;
    const uint32_t static_bytes = reinterpret_cast<const TabHdr*>(pp.blob)->static_bytes;
    if (!bulk_load(dyn, pp.blob, static_bytes, &mbar)) {
        if (tid == 0) atomicExch(&pp.ctrl->error, 1u);
        for (uint32_t x = tid; x < static_bytes / 16; x += PLAN_THREADS)
            reinterpret_cast<uint4*>(dyn)[x] = reinterpret_cast<const uint4*>(pp.blob)[x];
        __syncthreads();
    }
    TabView v;
    v.bind(dyn, pp.blob);
    finish_pass(pp, v, s_hits, reinterpret_cast<uint32_t*>(dyn + static_bytes), &s_n, n_partial);
}

// The tables of every configuration, built once per (context, space) and kept in global memory: all of them but
// the availability mask of the last segment depend on the context and the configuration only, so a search after
// a new snapshot copies them instead of rebuilding them.  One block per configuration at a time.
__global__ void __launch_bounds__(PLAN_THREADS, PLAN_MIN_BLOCKS) cfg_cache_kernel(const __grid_constant__ PlanParams pp, uint4* cache) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ CfgShared cs;
    const uint32_t tid = threadIdx.x;
    const TabHdr* gh = reinterpret_cast<const TabHdr*>(pp.blob);
    const uint32_t static_bytes = gh->static_bytes;
    if (!bulk_load(dyn, pp.blob, static_bytes, &cs.mbar)) {
        if (tid == 0) atomicExch(&pp.ctrl->error, 1u);
        for (uint32_t x = tid; x < static_bytes / 16; x += PLAN_THREADS)
            reinterpret_cast<uint4*>(dyn)[x] = reinterpret_cast<const uint4*>(pp.blob)[x];
        __syncthreads();
    }
    TabView v;
    v.bind(dyn, pp.blob);
    const uint32_t T = v.h->T, Z = v.h->Z;
    CfgArrays a;
    carve(dyn, static_bytes, pp.p_max, T, Z, a);
    // the whole cached region starts from zero, so that records do not depend on what the block did before
    for (uint32_t x = tid; x < pp.cache_arr16; x += PLAN_THREADS) reinterpret_cast<uint4*>(a.rec)[x] = make_uint4(0, 0, 0, 0);
    for (uint32_t x = tid; x < pp.cache_head16; x += PLAN_THREADS) reinterpret_cast<uint4*>(&cs)[x] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (uint32_t c = blockIdx.x; c < pp.n_config; c += gridDim.x) {
        __syncthreads();
        build_config(pp, v, cs, a, c);
        __syncthreads();
        uint4* dst = cache + (size_t)c * (pp.cache_head16 + pp.cache_arr16);
        for (uint32_t x = tid; x < pp.cache_head16; x += PLAN_THREADS) dst[x] = reinterpret_cast<const uint4*>(&cs)[x];
        for (uint32_t x = tid; x < pp.cache_arr16; x += PLAN_THREADS) dst[pp.cache_head16 + x] = reinterpret_cast<const uint4*>(a.rec)[x];
    }
}

// Which prefixes can matter at all?  Per configuration: the digits of every segment whose type can
// host tp and whose stages fit in memory (H2: independent of availability), hence the number of
// chunks of prefixes made of such digits only, and -- in closed form -- how many candidates are
// invalid or out of memory.  Runs once per (context, space); the plan search then enumerates only
// the live prefixes.  One block per configuration at a time.
constexpr int SURVEY_THREADS = 128;

__global__ void __launch_bounds__(SURVEY_THREADS)
survey_kernel(const unsigned char* __restrict__ blob, SpaceDesc sp, uint32_t n_config, uint32_t* __restrict__ live_chunks,
              unsigned long long* __restrict__ closed /* total, invalid, oom */,
              unsigned long long* __restrict__ cfg_closed /* [n_config][3], the same per configuration; may be null */) {
    __shared__ uint32_t oom_stage[SAILOR_P_MAX];
    __shared__ Config k;
    __shared__ uint32_t valid;
    __shared__ uint64_t n_b;
    TabView v;
    v.bind(blob, blob);
    const TabHdr* h = v.h;
    const uint32_t T = h->T, R = h->R, tid = threadIdx.x;
    for (uint32_t c = blockIdx.x; c < n_config; c += gridDim.x) {
        __syncthreads();
        if (tid == 0) {
            k = config_of(sp, c);
            const uint32_t tp = h->tp_values[k.tpi];
            const uint64_t dm = (uint64_t)k.D * h->mbs_values[k.mi];
            valid = (k.D >= 1 && h->gbs % dm == 0 && h->heads % tp == 0) ? 1u : 0u;
            n_b = k.D >= 1 ? h->gbs / dm : 0;
        }
        for (uint32_t i = tid; i < SAILOR_P_MAX; i += SURVEY_THREADS) oom_stage[i] = 0;
        __syncthreads();
        const uint32_t P = k.P;
        if (valid) {
            const uint32_t base = h->n_blocks / P, extra = h->n_blocks % P;
            for (uint32_t x = tid; x < P * T; x += SURVEY_THREADS) {
                const uint32_t i = x / T, g = x % T;
                const uint32_t nb = base + (i < extra ? 1u : 0u);
                const bool e = (i == 0) && h->has_embed, hd = (i == P - 1) && h->has_head;
                const uint64_t inflight = (uint64_t)(P - i) < n_b ? (uint64_t)(P - i) : n_b;
                const StageMem sm = stage_memory(v, k.tpi, k.mi, k.rc, nb, e, hd, inflight);
                if (sm.mem + h->reserved[g] > h->capacity[g]) atomicOr(&oom_stage[i], 1u << g);
            }
        }
        __syncthreads();
        if (tid == 0) {
            const uint64_t n_all = ipow64(R, k.nseg);
            uint32_t chunks = 0;
            unsigned long long mine[3] = {n_all, n_all, 0};     // total, invalid, oom of this configuration
            if (valid) {
                const uint32_t tp = h->tp_values[k.tpi];
                uint32_t type_ok = 0;                      // types whose nodes can host tp
                for (uint32_t g = 0; g < T; ++g)
                    if (tp <= h->gpn[g]) type_ok |= 1u << g;
                const uint64_t n_valid = ipow64((uint64_t)__popc(type_ok) * h->Z, k.nseg);
                uint64_t live = 1, fit = 1;
                for (uint32_t s = 0; s < k.nseg; ++s) {
                    const uint32_t sa = (s * P + k.nseg - 1) / k.nseg, se = ((s + 1) * P + k.nseg - 1) / k.nseg;
                    uint32_t oom = 0;
                    for (uint32_t i = sa; i < se; ++i) oom |= oom_stage[i];
                    const uint64_t g_cnt = (uint64_t)__popc(type_ok & ~oom) * h->Z;     // usable digits of the segment
                    fit *= g_cnt;
                    if (s + 1 < k.nseg) live *= g_cnt;
                }
                if (fit) chunks = (uint32_t)((live + PLAN_THREADS - 1) / PLAN_THREADS);
                mine[1] = n_all - n_valid;
                mine[2] = n_valid - fit;
            }
            for (int j = 0; j < 3; ++j) {
                if (mine[j]) atomicAdd(&closed[j], mine[j]);
                if (cfg_closed) cfg_closed[3 * (size_t)c + j] = mine[j];
            }
            live_chunks[c] = chunks;
        }
    }
}

// ---- searches in degree order (H3 / H4) -----------------------------------------------------------
//
// A group is a configuration without its data-parallel degree; its degrees sit next to each other in
// the configuration index (c = group * n_d + position in d_values).  The rule of a group is
// sequential (try the next degree only while the last one improved), but the groups are independent,
// so they advance together: wave w evaluates, for every group still going, the w-th degree of the
// order.  Between two waves one small block applies the rule to what the last wave found and lays
// out the chunk table of the next one; nothing returns to the host in between.
struct GroupState {
    unsigned long long prev_bits;      // best score at the last degree that had a feasible plan
    uint32_t state;                    // 0: no feasible degree yet, 1: going, 2: stopped
    uint32_t _pad;
};

struct WaveParams {
    const uint32_t* live_start;        // [n_config + 1] chunk offsets when every configuration is searched
    const unsigned long long* cfg_closed;   // [n_config][3] total, invalid, oom per configuration
    uint32_t* wave_start;              // [n_config + 1] out: chunk offsets of this wave
    unsigned long long* cfg_best;      // [n_config]
    GroupState* groups;                // [n_config / n_d]
    Ctrl* ctrl;
    uint32_t n_config, n_d, wave;
    uint8_t order[SAILOR_ND_MAX];      // positions in d_values, in the order they are tried
};

constexpr int WAVE_THREADS = 1024;

__global__ void __launch_bounds__(WAVE_THREADS) wave_step_kernel(const __grid_constant__ WaveParams wp) {
    __shared__ uint32_t warp_sum[WAVE_THREADS / 32];
    __shared__ unsigned long long s_closed[3];
    __shared__ uint32_t s_eval;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t n_groups = wp.n_config / wp.n_d;
    const unsigned long long inf_bits = (unsigned long long)__double_as_longlong(make_inf());
    if (tid < 3) s_closed[tid] = 0;
    if (tid == 0) s_eval = 0;
    // the rule, applied to what the previous wave found
    for (uint32_t g = tid; g < n_groups; g += WAVE_THREADS) {
        GroupState gs = wp.groups[g];
        if (wp.wave == 0) { gs.prev_bits = inf_bits; gs.state = 0; gs._pad = 0; }
        else if (gs.state != 2) {
            const unsigned long long best = wp.cfg_best[(size_t)g * wp.n_d + wp.order[wp.wave - 1]];
            if (best == inf_bits) { if (gs.state == 1) gs.state = 2; }         // nothing feasible at that degree
            else if (gs.state == 1 && !(best < gs.prev_bits)) gs.state = 2;     // no strict improvement
            else { gs.prev_bits = best; gs.state = 1; }
        }
        wp.groups[g] = gs;
    }
    __syncthreads();
    // chunk table of this wave: the configuration (group, order[wave]) of every group still going
    const uint32_t per = (wp.n_config + WAVE_THREADS - 1) / WAVE_THREADS;
    const uint32_t c0 = min(tid * per, wp.n_config), c1 = min(c0 + per, wp.n_config);
    const uint32_t pick = wp.order[wp.wave];
    uint32_t mine = 0, n_eval = 0;
    unsigned long long closed[3] = {0, 0, 0};
    for (uint32_t c = c0; c < c1; ++c) {
        if (c % wp.n_d != pick || wp.groups[c / wp.n_d].state == 2) continue;
        mine += wp.live_start[c + 1] - wp.live_start[c];
        wp.cfg_best[c] = inf_bits;
        ++n_eval;
        for (int j = 0; j < 3; ++j) closed[j] += wp.cfg_closed[3 * (size_t)c + j];
    }
    uint32_t incl = mine;                                   // exclusive scan of `mine` over the block
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(FULL, incl, o);
        if (lane >= (uint32_t)o) incl += up;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = warp_sum[lane], wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(FULL, wi, o);
            if (lane >= (uint32_t)o) wi += up;
        }
        warp_sum[lane] = wi - w;
        if (lane == 31) {
            wp.wave_start[wp.n_config] = wi;
            wp.ctrl->wave_chunks = wi;
            wp.ctrl->work_counter = 0;
        }
    }
    __syncthreads();
    uint32_t at = warp_sum[warp] + incl - mine;
    for (uint32_t c = c0; c < c1; ++c) {
        wp.wave_start[c] = at;
        if (c % wp.n_d == pick && wp.groups[c / wp.n_d].state != 2) at += wp.live_start[c + 1] - wp.live_start[c];
    }
    for (int j = 0; j < 3; ++j)
        if (closed[j]) atomicAdd(&s_closed[j], closed[j]);
    if (n_eval) atomicAdd(&s_eval, n_eval);
    __syncthreads();
    if (tid < 3 && s_closed[tid]) atomicAdd(&wp.ctrl->stats[tid], s_closed[tid]);
    if (tid == 0) wp.ctrl->n_cfg_evaluated += s_eval;
}

}  // namespace sailor
