// C ABI of the library (see include/sailor.h): context management, argument checks, launches.
// Every simulation step runs in the kernels; the host only validates, packs tables and
// enqueues work on the caller's stream.
#include <atomic>
#include <cmath>
#include <cstddef>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <algorithm>
#include <array>
#include <map>

#include "sailor_batch.cuh"
#include "sailor_dp.cuh"
#include "sailor_dp_budget.cuh"
#include "sailor_mixed.cuh"
#include "sailor_mixed_search.cuh"
#include "sailor_peaks.cuh"

using namespace sailor;

namespace {

constexpr int SIM_THREADS = 256;
constexpr int PLAN_SMEM_CEILING = 200 * 1024;    // dynamic shared memory any search may ask for

// ---- kernels of the explicit-batch path -----------------------------------------------------

// Left-to-right layer sums for every stage composition: chain[n] = start + n blocks, where
// start is 0 or the embedding layer's entry.  One thread per (table, start, type, tp[, mbs]).
__global__ void chain_kernel(unsigned char* blob) {
    TabView v;
    v.bind(blob, blob);
    const TabHdr* h = v.h;
    const uint32_t gts = h->T * h->n_tp;
    const uint32_t n4 = 2 * gts * h->n_mbs;                  // [start][type][tp][mbs]
    const uint32_t n3 = 2 * gts;                             // [start][type][tp]
    const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x < 2 * n4) {
        const bool is_b = x >= n4;
        const uint32_t y = is_b ? x - n4 : x;
        const uint32_t mi = y % h->n_mbs, gt = (y / h->n_mbs) % gts, start = y / (h->n_mbs * gts);
        const double* tab = is_b ? v.bwd : v.fwd;
        double* out = reinterpret_cast<double*>(blob + (is_b ? h->off_chain_b : h->off_chain_f)) + (size_t)y * h->chain_len;
        const double e = tab[((size_t)KIND_EMBED * gts + gt) * h->n_mbs + mi];
        const double b = tab[((size_t)KIND_BLOCK * gts + gt) * h->n_mbs + mi];
        double acc = start ? add_rn(0.0, e) : 0.0;
        out[0] = acc;
        for (uint32_t n = 1; n < h->chain_len; ++n) { acc = add_rn(acc, b); out[n] = acc; }
    } else if (x < 2 * n4 + n3) {
        const uint32_t y = x - 2 * n4;
        const uint32_t gt = y % gts, start = y / gts;
        double* out = reinterpret_cast<double*>(blob + h->off_chain_u) + (size_t)y * h->chain_len;
        const double e = v.upd[(size_t)KIND_EMBED * gts + gt];
        const double b = v.upd[(size_t)KIND_BLOCK * gts + gt];
        double acc = start ? add_rn(0.0, e) : 0.0;
        out[0] = acc;
        for (uint32_t n = 1; n < h->chain_len; ++n) { acc = add_rn(acc, b); out[n] = acc; }
    }
}

// What a stage needs, per stage composition (embedding?, head?, number of blocks): parameters, gradient bytes per
// worker, memory without and per in-flight microbatch, f + b, update time.  Formed with the same functions and
// the same operation order as a stage-by-stage evaluation; one thread per (composition, type, tp, mbs, rc).
__global__ void compose_kernel(unsigned char* blob) {
    TabView v;
    v.bind(blob, blob);
    const TabHdr* h = v.h;
    const size_t n_comp = (size_t)4 * h->chain_len;
    const size_t total = n_comp * h->T * h->n_tp * h->n_mbs * 2;
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
        reinterpret_cast<double*>(blob + h->off_cmp_fb)[x] = add_rn(st.f, b);
        if (mi == 0 && rc == 0) reinterpret_cast<double*>(blob + h->off_cmp_upd)[(comp * h->T + g) * h->n_tp + tpi] = st.u;
        if (g == 0) {
            const StageMem one = stage_memory(v, tpi, mi, rc, nb, e, hd, 1);     // model + 1 * kept + work
            const StageMem zero = stage_memory(v, tpi, mi, rc, nb, e, hd, 0);    // model + work
            uint64_t* mm = reinterpret_cast<uint64_t*>(blob + h->off_cmp_mem) + (((comp * h->n_tp + tpi) * h->n_mbs + mi) * 2 + rc) * 2;
            mm[0] = zero.mem;
            mm[1] = one.mem - zero.mem;
            if (mi == 0 && rc == 0) {
                reinterpret_cast<double*>(blob + h->off_cmp_grad)[comp * h->n_tp + tpi] =
                    (double)(ceil_div64(one.params, h->tp_values[tpi]) * h->grad_bytes);
                if (tpi == 0) reinterpret_cast<uint64_t*>(blob + h->off_cmp_params)[comp] = one.params;
            }
        }
    }
}

// One warp per plan with mixed replicas (records `stride` bytes apart holding `max_stages` stages, read in place,
// lane i reading stage i).  Tables in shared memory, then R 64-bit GPU counters per warp.  Plans of up to 32 stages
// are evaluated by the DEEP = false launch, which leaves deeper ones alone and notes in `deep_seen` that there are
// some; the DEEP = true launch that follows returns at once when there are none and evaluates only those otherwise
// (a lane then owns up to three stages; the state of that evaluation does not fit the registers of the first).
template <bool DEEP>
__global__ void __launch_bounds__(SIM_THREADS, DEEP ? 2 : 4)
simulate_mixed_kernel(const unsigned char* __restrict__ blob, const uint16_t* __restrict__ avail,
                      const unsigned char* __restrict__ plans, uint32_t stride, uint32_t max_stages, uint64_t n,
                      double* __restrict__ t_iter, uint64_t* __restrict__ peak_mem, double* __restrict__ cost,
                      uint32_t* __restrict__ status, unsigned int* error, unsigned int* deep_seen, uint32_t report_bad) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ uint64_t mbar;
    if (DEEP && *reinterpret_cast<volatile unsigned int*>(deep_seen) == 0) return;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    constexpr uint32_t WARPS = SIM_THREADS / 32;
    const uint32_t static_bytes = reinterpret_cast<const TabHdr*>(blob)->static_bytes;
    if (!bulk_load(dyn, blob, static_bytes, &mbar)) {
        if (tid == 0) atomicOr(error, SIM_ERR_DEVICE);
        for (uint32_t x = tid; x < static_bytes / 16; x += SIM_THREADS)
            reinterpret_cast<uint4*>(dyn)[x] = reinterpret_cast<const uint4*>(blob)[x];
        __syncthreads();
    }
    TabView v;
    v.bind(dyn, blob);
    unsigned long long* counters = reinterpret_cast<unsigned long long*>(dyn + static_bytes) + (size_t)warp * v.h->R;
    for (uint64_t j = (uint64_t)blockIdx.x * WARPS + warp; j < n; j += (uint64_t)gridDim.x * WARPS) {
        const sailor_mixed_plan& r = *reinterpret_cast<const sailor_mixed_plan*>(plans + j * stride);
        const uint32_t P = r.P;
        SimOut o;
        if (DEEP) {
            if (P <= 32 || P > max_stages) continue;             // done by the first launch
            o = simulate_mixed_tiles<SAILOR_MIX_P_MAX / 32>(v, avail, r, counters, lane);
        } else if (P > max_stages) {                             // more stages than the record has room for
            o.t_iter = o.cost = make_nan();
            o.peak_mem = 0;
            o.status = SAILOR_ST_BAD_RECORD;
        } else if (P > 32) {
            if (lane == 0) *reinterpret_cast<volatile unsigned int*>(deep_seen) = 1u;
            continue;
        } else {
            o = simulate_mixed_warp(v, avail, r, counters, lane);
        }
        if (lane == 0) {
            if (t_iter) t_iter[j] = o.t_iter;
            if (peak_mem) peak_mem[j] = o.peak_mem;
            if (cost) cost[j] = o.cost;
            if (status) status[j] = o.status;
            if (report_bad && (o.status & SAILOR_ST_BAD_RECORD)) atomicOr(error, SIM_ERR_BAD_RECORD);
        }
        __syncwarp();
    }
}

// ---- host state -----------------------------------------------------------------------------

struct SpaceCache {
    bool valid = false;
    sailor_space key;
    SpaceDesc desc;
    uint32_t n_config = 0, n_chunks = 0, p_max = 0;
    uint64_t n_total = 0;
    std::vector<uint32_t> chunk_start;     // host copies, for range -> chunk lookup
    std::vector<uint64_t> flat_base;
    uint32_t* d_chunk_start = nullptr;
    uint64_t* d_flat_base = nullptr;
    size_t smem = 0, smem_screen = 0;      // dynamic shared memory of a search block, without and with the binary32 tables
    // chunks of live prefixes only (see survey_kernel), for whole-space searches with pruning on
    uint32_t* d_live_start = nullptr;      // [n_config + 1]
    uint32_t live_chunks = 0;
    unsigned long long closed[3] = {0, 0, 0};   // candidates counted in closed form: total, invalid, oom
    // searches in degree order (spaces of at most WAVE_CONFIG_MAX configurations)
    unsigned long long* d_cfg_closed = nullptr;   // [n_config][3] the closed-form counts per configuration
    uint32_t* d_wave_start = nullptr;             // [n_config + 1] chunk offsets of the current wave
    unsigned long long* d_cfg_best = nullptr;     // [n_config] best feasible score per configuration
    GroupState* d_groups = nullptr;               // [n_config / n_d]
    // the per-configuration tables, built once per space (spaces whose records fit CFG_CACHE_MAX_BYTES)
    uint4* d_cfg_cache = nullptr;
    uint32_t cache_head16 = 0, cache_arr16 = 0;
};

constexpr size_t CFG_CACHE_MAX_BYTES = 512ull << 20;

constexpr uint64_t WAVE_CONFIG_MAX = 1u << 16;

}  // namespace

static_assert(offsetof(Ctrl, thr_bits) == offsetof(Ctrl, min_cost_bits) + 8, "cleared together");

struct sailor_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int last_cuda = 0;
    int sm_count = 0;
    TabHdr hdr;                            // host copy of the header
    unsigned char* d_blob = nullptr;
    uint16_t* d_avail = nullptr;           // device copy for the kernels that take a pointer (brought up to date lazily)
    uint16_t* h_avail = nullptr;           // pinned; the snapshot last set
    bool avail_dirty = false;              // d_avail is older than h_avail
    PlanOut* d_out_mapped = nullptr;       // device address of h_out (mapped pinned memory)
    Ctrl* d_ctrl = nullptr;
    unsigned int* d_sim_error = nullptr;   // error word of the explicit-batch kernels, then the "deep plans seen" word
    PlanOut* h_out = nullptr;              // pinned
    bool ctrl_dirty = true;                // the counters must be cleared from the host (first call, or after a failed one)
    uint64_t sync_epoch = 1;               // stream synchronisations by this context so far
    uint64_t avail_epoch = 0;              // sync_epoch when the pinned availability buffer was last handed to a copy
    bool h2d_fresh = false;                // an availability upload has been timed and not yet read
    float h2d_ms = 0.f;
    Hit* d_partial = nullptr;
    uint32_t* d_partial_n = nullptr;
    uint32_t max_grid = 0;                 // capacity of the partial-result buffers
    uint32_t grid_of[15] = {0};            // resident blocks per kernel variant, for the cached space
    SpaceCache space;
    cudaEvent_t ev0 = nullptr, ev1 = nullptr, ev2 = nullptr, evh0 = nullptr, evh1 = nullptr;
    cudaStream_t out_stream = nullptr;     // results of a host batch leave on it while the next chunk comes in
    cudaEvent_t ev_chunk = nullptr, ev_join = nullptr, ev_slot[3] = {nullptr, nullptr, nullptr};
    // explicit-batch staging (grow-only)
    unsigned char* d_stage = nullptr;
    size_t stage_bytes = 0;
    // working memory of the search over plans with mixed replicas (grow-only)
    unsigned char* d_mix = nullptr;
    size_t mix_bytes = 0;
    // tables of the dynamic-programming search (grow-only)
    unsigned char* d_dp = nullptr;
    size_t dp_bytes = 0;
};

namespace {

#define CU(ctx, call)                                  \
    do {                                               \
        cudaError_t e_ = (call);                       \
        if (e_ != cudaSuccess) {                       \
            (ctx)->last_cuda = (int)e_;                \
            return SAILOR_E_CUDA;                      \
        }                                              \
    } while (0)

// Synchronise the context's stream; everything enqueued before (the availability upload among it) is done after.
cudaError_t stream_sync(sailor_ctx* ctx) {
    const cudaError_t e = cudaStreamSynchronize(ctx->stream);
    if (e == cudaSuccess) ++ctx->sync_epoch;
    return e;
}

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        cudaGetDevice(&prev);
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

bool finite_nonneg(const double* p, size_t n) {
    for (size_t i = 0; i < n; ++i)
        if (!(p[i] >= 0.0) || std::isinf(p[i])) return false;
    return true;
}

uint32_t align16(uint32_t x) { return (x + 15u) & ~15u; }

template <typename T>
uint32_t put(std::vector<unsigned char>& blob, const T* src, size_t n) {
    const uint32_t off = align16((uint32_t)blob.size());
    blob.resize(off + n * sizeof(T));
    if (src) memcpy(blob.data() + off, src, n * sizeof(T));
    return off;
}

int check_space(const sailor_ctx* ctx, const sailor_space* s) {
    if (!ctx || !s) return SAILOR_E_ARG;
    if (s->n_p == 0 || s->n_mbs == 0 || s->n_tp == 0 || s->n_rc == 0 || s->n_d == 0) return SAILOR_E_ARG;
    if (s->n_p > SAILOR_NP_MAX || s->n_mbs > SAILOR_MBS_MAX || s->n_tp > SAILOR_TP_MAX || s->n_rc > 2 ||
        s->n_d > SAILOR_ND_MAX || s->seg_max < 1 || s->seg_max > SAILOR_SEG_MAX)
        return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < s->n_p; ++i)
        if (s->p_values[i] < 1 || s->p_values[i] > SAILOR_P_MAX) return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < s->n_mbs; ++i)
        if (s->mbs_idx[i] >= ctx->hdr.n_mbs) return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < s->n_tp; ++i)
        if (s->tp_idx[i] >= ctx->hdr.n_tp) return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < s->n_rc; ++i)
        if (s->rc_values[i] > 1) return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < s->n_d; ++i)
        if (s->d_values[i] < 1) return SAILOR_E_RANGE;
    return SAILOR_OK;
}

SpaceDesc to_desc(const sailor_space* s) {
    SpaceDesc d;
    memset(&d, 0, sizeof(d));
    d.n_p = s->n_p; d.n_mbs = s->n_mbs; d.n_tp = s->n_tp; d.n_rc = s->n_rc; d.n_d = s->n_d; d.seg_max = s->seg_max;
    memcpy(d.p_values, s->p_values, sizeof(d.p_values));
    memcpy(d.mbs_idx, s->mbs_idx, sizeof(d.mbs_idx));
    memcpy(d.tp_idx, s->tp_idx, sizeof(d.tp_idx));
    memcpy(d.rc_values, s->rc_values, sizeof(d.rc_values));
    memcpy(d.d_values, s->d_values, sizeof(d.d_values));
    return d;
}

// Candidate count with overflow check (limit 2^63).
int space_total(const sailor_ctx* ctx, const SpaceDesc& d, uint64_t* out) {
    const uint64_t R = ctx->hdr.R;
    const uint64_t base = (uint64_t)d.n_mbs * d.n_tp * d.n_rc * d.n_d;
    unsigned __int128 n = 0;
    for (uint32_t j = 0; j < d.n_p; ++j) {
        n += (unsigned __int128)base * ipow64(R, nseg_of(d.p_values[j], d.seg_max));
        if (n >> 63) return SAILOR_E_RANGE;
    }
    *out = (uint64_t)n;
    return SAILOR_OK;
}

bool same_space(const sailor_space& a, const sailor_space& b) {
    if (a.n_p != b.n_p || a.n_mbs != b.n_mbs || a.n_tp != b.n_tp || a.n_rc != b.n_rc || a.n_d != b.n_d ||
        a.seg_max != b.seg_max)
        return false;
    return !memcmp(a.p_values, b.p_values, a.n_p) && !memcmp(a.mbs_idx, b.mbs_idx, a.n_mbs) &&
           !memcmp(a.tp_idx, b.tp_idx, a.n_tp) && !memcmp(a.rc_values, b.rc_values, a.n_rc) &&
           !memcmp(a.d_values, b.d_values, a.n_d * sizeof(uint16_t));
}

// Per-configuration chunk and flat-index offsets; uploaded once per distinct space.
int prepare_space(sailor_ctx* ctx, const sailor_space* s) {
    SpaceCache& sc = ctx->space;
    if (sc.valid && same_space(sc.key, *s)) return SAILOR_OK;
    int rc = check_space(ctx, s);
    if (rc) return rc;
    SpaceDesc d = to_desc(s);
    uint64_t total = 0;
    rc = space_total(ctx, d, &total);
    if (rc) return rc;
    const uint64_t R = ctx->hdr.R;
    const uint32_t per_p = d.n_mbs * d.n_tp * d.n_rc * d.n_d;
    const uint64_t n_config = (uint64_t)per_p * d.n_p;
    if (n_config > (1u << 24)) return SAILOR_E_RANGE;
    std::vector<uint32_t> cs(n_config + 1);
    std::vector<uint64_t> fb(n_config);
    uint64_t chunks = 0, flat = 0;
    uint32_t p_max = 0;
    for (uint32_t j = 0; j < d.n_p; ++j) {
        const uint32_t nseg = nseg_of(d.p_values[j], d.seg_max);
        p_max = d.p_values[j] > p_max ? d.p_values[j] : p_max;
        const uint64_t items = ipow64(R, nseg - 1);
        const uint64_t per_cfg = (items + PLAN_THREADS - 1) / PLAN_THREADS;
        for (uint32_t c = 0; c < per_p; ++c) {
            cs[(size_t)j * per_p + c] = (uint32_t)chunks;
            fb[(size_t)j * per_p + c] = flat;
            chunks += per_cfg;
            flat += items * R;
            if (chunks >= 0xfff00000ull) return SAILOR_E_RANGE;
        }
    }
    cs[n_config] = (uint32_t)chunks;
    const size_t smem = plan_smem_bytes(ctx->hdr.static_bytes, p_max, ctx->hdr.T, ctx->hdr.Z, (uint32_t)n_config);
    if (smem > (size_t)PLAN_SMEM_CEILING) return SAILOR_E_RANGE;

    sc.valid = false;
    cudaFree(sc.d_chunk_start);
    cudaFree(sc.d_flat_base);
    sc.d_chunk_start = nullptr;
    sc.d_flat_base = nullptr;
    CU(ctx, cudaMalloc(&sc.d_chunk_start, cs.size() * sizeof(uint32_t)));
    CU(ctx, cudaMalloc(&sc.d_flat_base, fb.size() * sizeof(uint64_t)));
    CU(ctx, cudaMemcpyAsync(sc.d_chunk_start, cs.data(), cs.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(ctx, cudaMemcpyAsync(sc.d_flat_base, fb.data(), fb.size() * sizeof(uint64_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(ctx, stream_sync(ctx));       // the vectors are pageable
    {   // survey the space once: live chunks per configuration and the closed-form class counts
        cudaFree(sc.d_live_start);
        cudaFree(sc.d_cfg_closed);
        cudaFree(sc.d_wave_start);
        cudaFree(sc.d_cfg_best);
        cudaFree(sc.d_groups);
        cudaFree(sc.d_cfg_cache);
        sc.d_cfg_cache = nullptr;
        sc.d_live_start = nullptr;
        sc.d_cfg_closed = nullptr;
        sc.d_wave_start = nullptr;
        sc.d_cfg_best = nullptr;
        sc.d_groups = nullptr;
        unsigned long long* d_closed = nullptr;
        CU(ctx, cudaMalloc(&sc.d_live_start, (n_config + 1) * sizeof(uint32_t)));
        if (n_config <= WAVE_CONFIG_MAX) {
            CU(ctx, cudaMalloc(&sc.d_cfg_closed, n_config * 3 * sizeof(unsigned long long)));
            CU(ctx, cudaMalloc(&sc.d_wave_start, (n_config + 1) * sizeof(uint32_t)));
            CU(ctx, cudaMalloc(&sc.d_cfg_best, n_config * sizeof(unsigned long long)));
            CU(ctx, cudaMalloc(&sc.d_groups, (n_config / d.n_d) * sizeof(GroupState)));
        }
        CU(ctx, cudaMalloc(&d_closed, 3 * sizeof(unsigned long long)));
        cudaError_t e = cudaMemsetAsync(d_closed, 0, 3 * sizeof(unsigned long long), ctx->stream);
        const uint32_t grid = (uint32_t)(n_config < 2048 ? n_config : 2048);
        if (e == cudaSuccess) {
            survey_kernel<<<grid, SURVEY_THREADS, 0, ctx->stream>>>(ctx->d_blob, d, (uint32_t)n_config, sc.d_live_start, d_closed,
                                                                    sc.d_cfg_closed);
            e = cudaGetLastError();
        }
        std::vector<uint32_t> live(n_config + 1, 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(live.data(), sc.d_live_start, n_config * sizeof(uint32_t), cudaMemcpyDeviceToHost, ctx->stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(sc.closed, d_closed, sizeof(sc.closed), cudaMemcpyDeviceToHost, ctx->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
        cudaFree(d_closed);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SAILOR_E_CUDA; }
        uint64_t run = 0;                              // exclusive scan on the host: once per space
        for (uint64_t j = 0; j < n_config; ++j) { const uint32_t v = live[j]; live[j] = (uint32_t)run; run += v; }
        live[n_config] = (uint32_t)run;
        sc.live_chunks = (uint32_t)run;
        CU(ctx, cudaMemcpyAsync(sc.d_live_start, live.data(), (n_config + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice, ctx->stream));
        CU(ctx, stream_sync(ctx));
    }
    {   // the tables of every configuration, once: later searches copy them instead of building them
        sc.cache_head16 = cache_head16();
        sc.cache_arr16 = cache_arr16(ctx->hdr.T, ctx->hdr.Z);
        const size_t rec_bytes = 16 * ((size_t)sc.cache_head16 + sc.cache_arr16);
        if (n_config * rec_bytes <= CFG_CACHE_MAX_BYTES && cudaMalloc(&sc.d_cfg_cache, n_config * rec_bytes) == cudaSuccess) {
            // (setting the attribute twice from two threads is harmless: both set the same value)
            static std::atomic<bool> optin_done[64];
            const bool tracked = ctx->device >= 0 && ctx->device < 64;
            if (!tracked || !optin_done[ctx->device].load(std::memory_order_acquire)) {
                CU(ctx, cudaFuncSetAttribute(cfg_cache_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PLAN_SMEM_CEILING));
                if (tracked) optin_done[ctx->device].store(true, std::memory_order_release);
            }
            PlanParams pp;
            memset(&pp, 0, sizeof(pp));
            pp.blob = ctx->d_blob;
            memcpy(pp.avail, ctx->h_avail, sizeof(pp.avail));
            pp.ctrl = ctx->d_ctrl;
            pp.cfg_flat_base = sc.d_flat_base;
            pp.sp = d;
            pp.n_config = (uint32_t)n_config;
            pp.p_max = p_max;
            pp.live_mode = 1;                  // the lists of usable digits are part of a record
            pp.min_tp_only = 1;                // and so are the masks of the smaller tensor-parallel degrees
            pp.cache_head16 = sc.cache_head16;
            pp.cache_arr16 = sc.cache_arr16;
            const uint32_t grid = (uint32_t)(n_config < (uint64_t)ctx->sm_count * 2 ? n_config : (uint64_t)ctx->sm_count * 2);
            cfg_cache_kernel<<<grid, PLAN_THREADS, smem, ctx->stream>>>(pp, sc.d_cfg_cache);
            CU(ctx, cudaGetLastError());
            CU(ctx, stream_sync(ctx));
        } else {
            sc.d_cfg_cache = nullptr;          // too large (or no memory): searches build the tables themselves
            (void)cudaGetLastError();
        }
    }
    sc.key = *s;
    sc.desc = d;
    sc.n_config = (uint32_t)n_config;
    sc.n_chunks = (uint32_t)chunks;
    sc.n_total = total;
    sc.p_max = p_max;
    sc.chunk_start.swap(cs);
    sc.flat_base.swap(fb);
    sc.smem = smem;
    sc.smem_screen = plan_smem_bytes(ctx->hdr.static_bytes, p_max, ctx->hdr.T, ctx->hdr.Z, (uint32_t)n_config, true);
    sc.valid = true;
    for (uint32_t& g : ctx->grid_of) g = 0;
    return SAILOR_OK;
}

// Chunk that contains flat index f (f < n_total).
uint32_t chunk_of(const sailor_ctx* ctx, uint64_t f) {
    const SpaceCache& sc = ctx->space;
    uint32_t lo = 0, hi = sc.n_config;
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) / 2;
        if (sc.flat_base[mid] <= f) lo = mid; else hi = mid;
    }
    const uint64_t item = (f - sc.flat_base[lo]) / ctx->hdr.R;
    return sc.chunk_start[lo] + (uint32_t)(item / PLAN_THREADS);
}

using PlanKernel = void (*)(const PlanParams);

constexpr int PLAN_VARIANTS = 15;      // objective x constraint x fused, then the three screened kernels

uint32_t variant_of(uint32_t obj, bool constr, bool fused, bool screen = false) {
    return screen ? 12 + obj : (obj * 2 + (constr ? 1 : 0)) * 2 + (fused ? 1 : 0);
}

template <bool FUSED>
PlanKernel pick_kernel_of(uint32_t obj, bool constr) {
    switch (obj) {
        case SAILOR_OBJ_MAX_THROUGHPUT: return constr ? plan_kernel<0, true, FUSED> : plan_kernel<0, false, FUSED>;
        case SAILOR_OBJ_MIN_COST: return constr ? plan_kernel<1, true, FUSED> : plan_kernel<1, false, FUSED>;
        default: return constr ? plan_kernel<2, true, FUSED> : plan_kernel<2, false, FUSED>;
    }
}

PlanKernel pick_kernel(uint32_t obj, bool constr, bool fused, bool screen = false) {
    if (screen)        // unconstrained searches only; they end their pass in finish_kernel
        return obj == SAILOR_OBJ_MAX_THROUGHPUT ? plan_kernel<0, false, false, true>
               : obj == SAILOR_OBJ_MIN_COST     ? plan_kernel<1, false, false, true>
                                                : plan_kernel<2, false, false, true>;
    return fused ? pick_kernel_of<true>(obj, constr) : pick_kernel_of<false>(obj, constr);
}

// Searches of up to this many chunks per resident block end their pass inside the search kernel; longer ones
// launch finish_kernel after it.
constexpr uint32_t FUSED_CHUNKS_PER_BLOCK = 256;

// The dynamic shared-memory opt-in belongs to the kernel (per device), not to a context: raise it
// once per (device, variant) to the ceiling every space is checked against, so that contexts
// with different table sizes cannot lower it under one another.
// The flags are atomic: contexts on different host threads may get here together, and setting the
// attribute twice to the same value is harmless.
std::atomic<bool> g_optin_done[64][PLAN_VARIANTS];

int smem_optin(sailor_ctx* ctx, PlanKernel kern, uint32_t variant) {
    const bool tracked = ctx->device >= 0 && ctx->device < 64;
    if (tracked && g_optin_done[ctx->device][variant].load(std::memory_order_acquire)) return SAILOR_OK;
    CU(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PLAN_SMEM_CEILING));
    if (tracked) g_optin_done[ctx->device][variant].store(true, std::memory_order_release);
    return SAILOR_OK;
}

// Enqueue one search pass on the context's stream: the search kernel, whose last block also merges the
// blocks' lists and writes the results (no separate merge launch, no clearing from the host).
//
// With SAILOR_FLAG_DEGREE_ORDER (whole space, live layout) the search runs as n_d waves: a one-block
// step kernel applies the H3/H4 rule to the previous wave's per-configuration bests and lays out the
// next wave's chunks, then the search kernel evaluates them; every block carries its list from wave
// to wave, and the last wave's launch ends the pass.
int enqueue_pass(sailor_ctx* ctx, uint32_t obj, double budget, bool budget_from_ctrl, double min_rate,
                 uint32_t flags, uint64_t lo, uint64_t hi, bool live, uint32_t k, double next_budget_factor,
                 uint32_t* n_launches, bool* launched) {
    SpaceCache& sc = ctx->space;
    const bool waves = (flags & SAILOR_FLAG_DEGREE_ORDER) != 0;
    // the counters start from the values the last finished pass (or the host, after a failure) left them at
    PlanParams pp;
    memset(&pp, 0, sizeof(pp));
    pp.blob = ctx->d_blob;
    memcpy(pp.avail, ctx->h_avail, sizeof(pp.avail));
    pp.cfg_chunk_start = sc.d_chunk_start;
    pp.cfg_flat_base = sc.d_flat_base;
    pp.ctrl = ctx->d_ctrl;
    pp.partial = ctx->d_partial;
    pp.partial_n = ctx->d_partial_n;
    pp.sp = sc.desc;
    pp.n_config = sc.n_config;
    pp.flat_lo = lo;
    pp.flat_hi = hi;
    pp.k = k;
    pp.eval_all = (flags & SAILOR_FLAG_EVAL_ALL) ? 1u : 0u;
    pp.min_tp_only = (flags & SAILOR_FLAG_MIN_TP_ONLY) ? 1u : 0u;
    pp.cfg_cache = sc.d_cfg_cache;
    pp.cache_head16 = sc.cache_head16;
    pp.cache_arr16 = sc.cache_arr16;
    pp.budget_from_ctrl = budget_from_ctrl ? 1u : 0u;
    pp.p_max = sc.p_max;
    pp.budget = budget;
    pp.min_rate = min_rate;
    pp.out = ctx->d_out_mapped;        // the block that ends the pass writes the results straight into pinned host memory
    pp.finish = 1;
    pp.next_budget_factor = next_budget_factor;
    pp.cost_only = next_budget_factor > 0.0 ? 1u : 0u;
    uint32_t grid = 0;
    if (waves) {                   // the chunk table and the chunk count of each wave are written on the device
        pp.cfg_chunk_start = sc.d_wave_start;
        pp.live_mode = 1;
        pp.chunk_lo = 0;
        pp.chunk_hi = 1;                           // the waves always run: they also gather the class counts
        pp.chunk_hi_dev = &ctx->d_ctrl->wave_chunks;
        pp.cfg_best = sc.d_cfg_best;
    } else if (live) {                    // whole space, pruning on: only chunks of live prefixes exist
        pp.cfg_chunk_start = sc.d_live_start;
        pp.live_mode = 1;
        pp.chunk_lo = 0;
        pp.chunk_hi = sc.live_chunks;
    } else if (hi > lo) {
        pp.chunk_lo = chunk_of(ctx, lo);
        pp.chunk_hi = chunk_of(ctx, hi - 1) + 1;
    }
    if (pp.chunk_hi > pp.chunk_lo) {
        const uint32_t n_chunks = waves ? sc.live_chunks : pp.chunk_hi - pp.chunk_lo;
        const bool constr = budget_from_ctrl || budget > 0.0 || min_rate > 0.0;
        const bool screen = (flags & SAILOR_FLAG_F32_SCREEN) != 0;
        const bool fused = !screen && n_chunks <= FUSED_CHUNKS_PER_BLOCK * 2u * (uint32_t)ctx->sm_count;
        PlanKernel kern = pick_kernel(obj, constr, fused, screen);
        const uint32_t variant = variant_of(obj, constr, fused, screen);
        const size_t smem_k = screen ? sc.smem_screen : sc.smem;
        if (smem_k > (size_t)PLAN_SMEM_CEILING) return SAILOR_E_RANGE;
        pp.screen = screen ? 1u : 0u;
        uint32_t& resident = ctx->grid_of[variant];
        if (resident == 0) {       // once per (space, kernel variant): size the grid
            int rc_opt = smem_optin(ctx, kern, variant);
            if (rc_opt) return rc_opt;
            int per_sm = 0;
            CU(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, PLAN_THREADS, smem_k));
            if (per_sm < 1) return SAILOR_E_RANGE;
            resident = (uint32_t)per_sm * (uint32_t)ctx->sm_count;
            if (resident > ctx->max_grid) resident = ctx->max_grid;
        }
        grid = n_chunks < resident ? (n_chunks ? n_chunks : 1u) : resident;
        const uint32_t batch = n_chunks / (grid * 32u);
        pp.batch = batch < 1 ? 1 : (batch > 16 ? 16 : batch);
        if (!waves) {
            kern<<<grid, PLAN_THREADS, smem_k, ctx->stream>>>(pp);
            CU(ctx, cudaGetLastError());
            ++*n_launches;
        } else {
            grid = resident < sc.live_chunks ? resident : (sc.live_chunks ? sc.live_chunks : 1u);   // the same blocks in every wave
            WaveParams wp;
            memset(&wp, 0, sizeof(wp));
            wp.live_start = sc.d_live_start;
            wp.cfg_closed = sc.d_cfg_closed;
            wp.wave_start = sc.d_wave_start;
            wp.cfg_best = sc.d_cfg_best;
            wp.groups = sc.d_groups;
            wp.ctrl = ctx->d_ctrl;
            wp.n_config = sc.n_config;
            wp.n_d = sc.desc.n_d;
            // H3: largest degree first when throughput is maximised; H4: smallest first when cost is minimised
            const bool descending = obj == SAILOR_OBJ_MAX_THROUGHPUT;
            for (uint32_t j = 0; j < wp.n_d; ++j) wp.order[j] = (uint8_t)j;
            for (uint32_t a = 1; a < wp.n_d; ++a) {        // stable insertion sort by degree
                const uint8_t x = wp.order[a];
                uint32_t b = a;
                while (b > 0 && (descending ? sc.desc.d_values[wp.order[b - 1]] < sc.desc.d_values[x]
                                            : sc.desc.d_values[wp.order[b - 1]] > sc.desc.d_values[x])) {
                    wp.order[b] = wp.order[b - 1];
                    --b;
                }
                wp.order[b] = x;
            }
            for (uint32_t w = 0; w < wp.n_d; ++w) {
                wp.wave = w;
                wave_step_kernel<<<1, WAVE_THREADS, 0, ctx->stream>>>(wp);
                CU(ctx, cudaGetLastError());
                pp.carry_lists = w ? 1u : 0u;
                pp.finish = (w + 1 == wp.n_d) ? 1u : 0u;       // the last wave's launch ends the pass
                kern<<<grid, PLAN_THREADS, sc.smem, ctx->stream>>>(pp);
                CU(ctx, cudaGetLastError());
                *n_launches += 2;
            }
        }
        if (!fused) {              // the end of the pass as a launch of its own
            finish_kernel<<<1, PLAN_THREADS, ctx->hdr.static_bytes + sizeof(uint32_t) * SAILOR_K_MAX * ctx->hdr.R, ctx->stream>>>(pp, grid);
            CU(ctx, cudaGetLastError());
            ++*n_launches;
        }
    }
    *launched = grid != 0;
    return SAILOR_OK;
}

// End of a host-side batch call: read the batch kernels' error word with the results, wait, and report (and
// clear) a fault.  Device-side batch calls only enqueue work; a fault in one of them is reported here as well,
// by the next host-side call.
int finish_host_batch(sailor_ctx* ctx) {
    unsigned int* h_err = &ctx->h_out->ctrl.error;               // pinned; no search is in flight on this context
    CU(ctx, cudaMemcpyAsync(h_err, ctx->d_sim_error, sizeof(unsigned int), cudaMemcpyDeviceToHost, ctx->stream));
    CU(ctx, stream_sync(ctx));
    if (*h_err) {
        CU(ctx, cudaMemsetAsync(ctx->d_sim_error, 0, sizeof(unsigned int), ctx->stream));
        return (*h_err & SIM_ERR_DEVICE) ? SAILOR_E_DEVICE : SAILOR_E_RANGE;
    }
    return SAILOR_OK;
}

// A host-side batch: records of `rec_bytes` in, four result arrays out (any may be NULL).  The batch goes through
// the device in chunks that take turns in HOST_SLOTS staging slots: a chunk's records are copied in and evaluated
// on the context's stream, its results leave on a second stream while the next chunk comes in, so that the two
// directions of the host link carry data at the same time; a slot is filled again only after its results have
// left.  The staging memory therefore does not grow with the batch beyond HOST_SLOTS chunks.  Records are checked
// by the kernel that reads them (`launch` passes the error word along, and a record outside its tables sets
// SIM_ERR_BAD_RECORD in it).  `launch(d_records, m, d_t, d_m, d_c, d_s)` enqueues the evaluation of m records on
// the context's stream.
constexpr uint64_t HOST_CHUNK_RECORDS = 1u << 19, HOST_CHUNK_BYTES = 1u << 26;
constexpr uint32_t HOST_SLOTS = 3;
int upload_availability(sailor_ctx* ctx);

template <class Launch>
int host_batch(sailor_ctx* ctx, const unsigned char* recs, size_t rec_bytes, uint64_t n, double* t_iter, uint64_t* peak_mem,
               double* cost, uint32_t* status, Launch launch) {
    uint64_t chunk = HOST_CHUNK_BYTES / rec_bytes;             // records per chunk: 64 MB of records, 2^19 at most
    chunk = chunk > HOST_CHUNK_RECORDS ? HOST_CHUNK_RECORDS : chunk;
    const bool split = n > chunk;
    const uint64_t slot_records = split ? chunk : n;
    const size_t slot_bytes = (slot_records * (rec_bytes + 32) + 255) / 256 * 256;
    const uint64_t n_chunks = (n + chunk - 1) / chunk;
    const size_t need = slot_bytes * (split ? (n_chunks < HOST_SLOTS ? n_chunks : HOST_SLOTS) : 1);
    if (need > ctx->stage_bytes) {
        CU(ctx, stream_sync(ctx));
        cudaFree(ctx->d_stage);
        ctx->d_stage = nullptr;
        ctx->stage_bytes = 0;
        cudaError_t e = cudaMalloc(&ctx->d_stage, need);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SAILOR_E_NOMEM; }
        ctx->stage_bytes = need;
    }
    {
        const int rc_up = upload_availability(ctx);
        if (rc_up) return rc_up;
    }
    cudaStream_t out = split ? ctx->out_stream : ctx->stream;
    int rc = SAILOR_OK;
    cudaError_t ce = cudaSuccess;
    uint64_t c = 0;
    for (uint64_t off = 0; off < n && ce == cudaSuccess && rc == SAILOR_OK; off += chunk, ++c) {
        const uint64_t m = n - off < chunk ? n - off : chunk;
        const uint32_t slot = (uint32_t)(c % HOST_SLOTS);
        unsigned char* base = ctx->d_stage + (split ? slot * slot_bytes : 0);
        double* d_t = reinterpret_cast<double*>(base);
        double* d_c = reinterpret_cast<double*>(base + 8 * slot_records);
        uint64_t* d_m = reinterpret_cast<uint64_t*>(base + 16 * slot_records);
        uint32_t* d_s = reinterpret_cast<uint32_t*>(base + 24 * slot_records);
        unsigned char* d_recs = base + 32 * slot_records;
        if (split && c >= HOST_SLOTS)                          // the slot's earlier results have to be out first
            if ((ce = cudaStreamWaitEvent(ctx->stream, ctx->ev_slot[slot], 0)) != cudaSuccess) break;
        ce = cudaMemcpyAsync(d_recs, recs + off * rec_bytes, m * rec_bytes, cudaMemcpyHostToDevice, ctx->stream);
        if (ce != cudaSuccess) break;
        rc = launch(d_recs, m, d_t, d_m, d_c, d_s);
        if (rc != SAILOR_OK) break;
        if (split) {
            if ((ce = cudaEventRecord(ctx->ev_chunk, ctx->stream)) != cudaSuccess) break;
            if ((ce = cudaStreamWaitEvent(out, ctx->ev_chunk, 0)) != cudaSuccess) break;
        }
        if (t_iter && ce == cudaSuccess) ce = cudaMemcpyAsync(t_iter + off, d_t, 8 * m, cudaMemcpyDeviceToHost, out);
        if (cost && ce == cudaSuccess) ce = cudaMemcpyAsync(cost + off, d_c, 8 * m, cudaMemcpyDeviceToHost, out);
        if (peak_mem && ce == cudaSuccess) ce = cudaMemcpyAsync(peak_mem + off, d_m, 8 * m, cudaMemcpyDeviceToHost, out);
        if (status && ce == cudaSuccess) ce = cudaMemcpyAsync(status + off, d_s, 4 * m, cudaMemcpyDeviceToHost, out);
        if (split && ce == cudaSuccess) ce = cudaEventRecord(ctx->ev_slot[slot], out);
    }
    if (split) {                   // whatever happened, the context's stream waits for what the second one was given
        cudaError_t cj = cudaEventRecord(ctx->ev_join, out);
        if (cj == cudaSuccess) cj = cudaStreamWaitEvent(ctx->stream, ctx->ev_join, 0);
        if (cj != cudaSuccess) { cudaStreamSynchronize(out); if (ce == cudaSuccess) ce = cj; }
    }
    const int rc_end = finish_host_batch(ctx);                 // waits for everything enqueued above
    if (ce != cudaSuccess) { ctx->last_cuda = (int)ce; return SAILOR_E_CUDA; }
    return rc != SAILOR_OK ? rc : rc_end;
}

// The device copy of the availability snapshot, for kernels that read it through a pointer.
int upload_availability(sailor_ctx* ctx) {
    if (!ctx->avail_dirty) return SAILOR_OK;
    CU(ctx, cudaEventRecord(ctx->evh0, ctx->stream));
    CU(ctx, cudaMemcpyAsync(ctx->d_avail, ctx->h_avail, ctx->hdr.R * sizeof(uint16_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(ctx, cudaEventRecord(ctx->evh1, ctx->stream));
    ctx->avail_epoch = ctx->sync_epoch;
    ctx->h2d_fresh = true;
    ctx->avail_dirty = false;
    return SAILOR_OK;
}

}  // namespace

// ---- C ABI ------------------------------------------------------------------------------------

extern "C" {

const char* sailor_strerror(int code) {
    switch (code) {
        case SAILOR_OK: return "ok";
        case SAILOR_E_ARG: return "invalid argument";
        case SAILOR_E_RANGE: return "index or size out of range";
        case SAILOR_E_CUDA: return "CUDA call failed";
        case SAILOR_E_NOMEM: return "out of memory";
        case SAILOR_E_DEVICE: return "kernel reported an internal fault";
        default: return "unknown error";
    }
}

int sailor_last_cuda_error(const sailor_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

static int create_impl(const sailor_model* m, const sailor_profile* p, const sailor_cluster* c, int cuda_device,
                       void* cuda_stream, sailor_ctx** out) {
    if (!m || !p || !c || !out) return SAILOR_E_ARG;
    *out = nullptr;
    if (!p->fwd || !p->bwd || !p->upd || !p->params || !p->act_saved || !p->act_ckpt || !p->act_work ||
        !p->p2p_bytes || !c->capacity || !c->reserved || !c->gpus_per_node || !c->price_per_hour ||
        !c->intra_alpha || !c->intra_inv_bw || !c->inter_alpha || !c->inter_inv_bw || !c->zone_alpha ||
        !c->zone_inv_bw || !c->egress)
        return SAILOR_E_ARG;
    const uint32_t T = p->n_types, Z = c->n_zones, n_tp = p->n_tp, n_mbs = p->n_mbs;
    if (T == 0 || Z == 0 || n_tp == 0 || n_mbs == 0 || T != c->n_types || m->n_blocks == 0) return SAILOR_E_ARG;
    if (m->gbs == 0 || m->heads == 0 || m->mul_factor == 0 || m->dtype_size == 0 || m->grad_dtype_size == 0)
        return SAILOR_E_ARG;
    if (T > SAILOR_T_MAX || Z > SAILOR_Z_MAX || n_tp > SAILOR_TP_MAX || n_mbs > SAILOR_MBS_MAX ||
        m->n_blocks > 4096)
        return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < n_tp; ++i)
        if (p->tp_values[i] == 0) return SAILOR_E_ARG;
    for (uint32_t i = 0; i < n_mbs; ++i)
        if (p->mbs_values[i] == 0) return SAILOR_E_ARG;
    for (uint32_t g = 0; g < T; ++g)
        if (c->gpus_per_node[g] == 0) return SAILOR_E_ARG;
    const size_t n4 = (size_t)SAILOR_KINDS * T * n_tp * n_mbs, n3 = (size_t)SAILOR_KINDS * T * n_tp;
    const size_t na = (size_t)SAILOR_KINDS * n_tp * n_mbs, R = (size_t)T * Z;
    if (!finite_nonneg(p->fwd, n4) || !finite_nonneg(p->bwd, n4) || !finite_nonneg(p->upd, n3) ||
        !finite_nonneg(c->price_per_hour, R) || !finite_nonneg(c->intra_alpha, R) ||
        !finite_nonneg(c->intra_inv_bw, R) || !finite_nonneg(c->inter_alpha, R) ||
        !finite_nonneg(c->inter_inv_bw, R) || !finite_nonneg(c->zone_alpha, (size_t)Z * Z) ||
        !finite_nonneg(c->zone_inv_bw, (size_t)Z * Z) || !finite_nonneg(c->egress, (size_t)Z * Z))
        return SAILOR_E_ARG;
    {   // bandwidth polynomials: coefficients finite and >= 0, constant term > 0 (bandwidth stays positive)
        const double* polys[3] = {c->intra_bw_poly, c->inter_bw_poly, c->zone_bw_poly};
        const size_t counts[3] = {R, R, (size_t)Z * Z};
        for (int q = 0; q < 3; ++q) {
            if (!polys[q]) continue;
            if (!finite_nonneg(polys[q], 4 * counts[q])) return SAILOR_E_ARG;
            for (size_t j = 0; j < counts[q]; ++j)
                if (!(polys[q][4 * j] > 0.0)) return SAILOR_E_ARG;
        }
    }

    sailor_ctx* ctx = new (std::nothrow) sailor_ctx();
    if (!ctx) return SAILOR_E_NOMEM;
    ctx->device = cuda_device;
    ctx->stream = (cudaStream_t)cuda_stream;
    DeviceGuard guard(cuda_device);

    // pack the blob: header, raw tables, cluster tables (static part), then the chains
    TabHdr& h = ctx->hdr;
    memset(&h, 0, sizeof(h));
    h.n_blocks = m->n_blocks; h.has_embed = m->has_embed ? 1 : 0; h.has_head = m->has_head ? 1 : 0;
    h.heads = m->heads; h.gbs = m->gbs;
    h.mul_bytes = (uint64_t)m->mul_factor * m->dtype_size;
    h.grad_bytes = m->grad_dtype_size;
    h.T = T; h.Z = Z; h.R = (uint32_t)R; h.n_tp = n_tp; h.n_mbs = n_mbs; h.chain_len = m->n_blocks + 1;
    memcpy(h.tp_values, p->tp_values, n_tp * sizeof(uint32_t));
    memcpy(h.mbs_values, p->mbs_values, n_mbs * sizeof(uint32_t));
    for (uint32_t g = 0; g < T; ++g) {
        h.gpn[g] = c->gpus_per_node[g];
        h.capacity[g] = c->capacity[g];
        h.reserved[g] = c->reserved[g];
    }
    for (int k = 0; k < SAILOR_KINDS; ++k) h.params[k] = p->params[k];
    for (uint32_t i = 0; i < n_tp; ++i)
        if (m->heads % p->tp_values[i] == 0) h.heads_ok |= 1u << i;

    std::vector<unsigned char> blob(sizeof(TabHdr));
    h.off_fwd = put(blob, p->fwd, n4);
    h.off_bwd = put(blob, p->bwd, n4);
    h.off_upd = put(blob, p->upd, n3);
    h.off_saved = put(blob, p->act_saved, na);
    h.off_ckpt = put(blob, p->act_ckpt, na);
    h.off_work = put(blob, p->act_work, na);
    h.off_p2p = put(blob, p->p2p_bytes, n_mbs);
    std::vector<double> price_s(R);
    for (size_t d = 0; d < R; ++d) price_s[d] = c->price_per_hour[d] / 3600.0;   // dollars per GPU-second
    h.off_price_s = put(blob, price_s.data(), R);
    h.off_intra_a = put(blob, c->intra_alpha, R);
    h.off_intra_i = put(blob, c->intra_inv_bw, R);
    h.off_inter_a = put(blob, c->inter_alpha, R);
    h.off_inter_i = put(blob, c->inter_inv_bw, R);
    h.off_zone_a = put(blob, c->zone_alpha, (size_t)Z * Z);
    h.off_zone_i = put(blob, c->zone_inv_bw, (size_t)Z * Z);
    h.off_egress = put(blob, c->egress, (size_t)Z * Z);
    h.off_intra_p = c->intra_bw_poly ? put(blob, c->intra_bw_poly, 4 * R) : 0;
    h.off_inter_p = c->inter_bw_poly ? put(blob, c->inter_bw_poly, 4 * R) : 0;
    h.off_zone_p = c->zone_bw_poly ? put(blob, c->zone_bw_poly, 4 * (size_t)Z * Z) : 0;
    h.static_bytes = align16((uint32_t)blob.size());
    blob.resize(h.static_bytes);
    const size_t c4 = (size_t)2 * T * n_tp * n_mbs * h.chain_len, c3 = (size_t)2 * T * n_tp * h.chain_len;
    const size_t n_comp = (size_t)4 * h.chain_len;
    const size_t cmp_fb = n_comp * T * n_tp * n_mbs * 2, cmp_upd = n_comp * T * n_tp, cmp_mem = n_comp * n_tp * n_mbs * 2 * 2,
                 cmp_grad = n_comp * n_tp;
    if (h.static_bytes + (2 * c4 + c3 + cmp_fb + cmp_upd + cmp_mem + cmp_grad + n_comp) * sizeof(double) +
                cmp_fb * sizeof(PieceRec) + (2 * R + (size_t)Z * Z) * n_mbs * sizeof(double) + 512 > (1ull << 30) ||
        h.static_bytes > 96 * 1024) {
        delete ctx;
        return SAILOR_E_RANGE;
    }
    h.off_chain_f = put<double>(blob, nullptr, c4);
    h.off_chain_b = put<double>(blob, nullptr, c4);
    h.off_chain_u = put<double>(blob, nullptr, c3);
    h.off_cmp_params = put<uint64_t>(blob, nullptr, n_comp);
    h.off_cmp_grad = put<double>(blob, nullptr, cmp_grad);
    h.off_cmp_mem = put<uint64_t>(blob, nullptr, cmp_mem);
    h.off_cmp_fb = put<double>(blob, nullptr, cmp_fb);
    h.off_cmp_upd = put<double>(blob, nullptr, cmp_upd);
    blob.resize((blob.size() + 31) & ~(size_t)31);         // a table entry is one 32-byte sector
    h.off_piece = put<PieceRec>(blob, nullptr, cmp_fb);
    h.off_lnk_intra2 = put<double>(blob, nullptr, R * n_mbs);
    h.off_lnk_inter2 = put<double>(blob, nullptr, R * n_mbs);
    h.off_lnk_zone2 = put<double>(blob, nullptr, (size_t)Z * Z * n_mbs);
    h.total_bytes = align16((uint32_t)blob.size());
    blob.resize(h.total_bytes);
    memcpy(blob.data(), &h, sizeof(h));

    auto fail = [&](int code) { sailor_destroy(ctx); return code; };
#define CUF(call)                                                   \
    do {                                                            \
        cudaError_t e_ = (call);                                    \
        if (e_ != cudaSuccess) {                                    \
            ctx->last_cuda = (int)e_;                               \
            return fail(e_ == cudaErrorMemoryAllocation ? SAILOR_E_NOMEM : SAILOR_E_CUDA); \
        }                                                           \
    } while (0)
    cudaDeviceProp prop;
    CUF(cudaGetDeviceProperties(&prop, cuda_device));
    ctx->sm_count = prop.multiProcessorCount;
    ctx->max_grid = (uint32_t)ctx->sm_count * 8;
    CUF(cudaMalloc(&ctx->d_blob, h.total_bytes));
    CUF(cudaMalloc(&ctx->d_avail, R_MAX * sizeof(uint16_t)));
    CUF(cudaMallocHost(&ctx->h_avail, R_MAX * sizeof(uint16_t)));
    memset(ctx->h_avail, 0, R_MAX * sizeof(uint16_t));       // availability starts at zero on both sides
    CUF(cudaMalloc(&ctx->d_ctrl, sizeof(Ctrl)));
    CUF(cudaMalloc(&ctx->d_sim_error, 2 * sizeof(unsigned int)));
    CUF(cudaHostAlloc(&ctx->h_out, sizeof(PlanOut), cudaHostAllocMapped));
    CUF(cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->d_out_mapped), ctx->h_out, 0));
    memset(ctx->h_out, 0, sizeof(PlanOut));
    CUF(cudaMalloc(&ctx->d_partial, sizeof(Hit) * SAILOR_K_MAX * ctx->max_grid));
    CUF(cudaMalloc(&ctx->d_partial_n, sizeof(uint32_t) * ctx->max_grid));
    CUF(cudaEventCreate(&ctx->ev0));
    CUF(cudaEventCreate(&ctx->ev1));
    CUF(cudaEventCreate(&ctx->ev2));
    CUF(cudaEventCreate(&ctx->evh0));
    CUF(cudaEventCreate(&ctx->evh1));
    CUF(cudaStreamCreateWithFlags(&ctx->out_stream, cudaStreamNonBlocking));
    CUF(cudaEventCreateWithFlags(&ctx->ev_chunk, cudaEventDisableTiming));
    CUF(cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming));
    for (cudaEvent_t& e : ctx->ev_slot) CUF(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    CUF(cudaMemcpyAsync(ctx->d_blob, blob.data(), h.total_bytes, cudaMemcpyHostToDevice, ctx->stream));
    CUF(cudaMemsetAsync(ctx->d_avail, 0, R_MAX * sizeof(uint16_t), ctx->stream));
    CUF(cudaMemsetAsync(ctx->d_ctrl, 0, sizeof(Ctrl), ctx->stream));
    CUF(cudaMemsetAsync(ctx->d_sim_error, 0, 2 * sizeof(unsigned int), ctx->stream));
    {
        const uint32_t n_threads = 4 * T * n_tp * n_mbs + 2 * T * n_tp;
        chain_kernel<<<(n_threads + 127) / 128, 128, 0, ctx->stream>>>(ctx->d_blob);
        CUF(cudaGetLastError());
        const size_t n_cmp = cmp_fb;
        const uint32_t grid = (uint32_t)((n_cmp + 127) / 128 < 65536 ? (n_cmp + 127) / 128 : 65536);
        compose_kernel<<<grid, 128, 0, ctx->stream>>>(ctx->d_blob);
        CUF(cudaGetLastError());
        batch_tables_kernel<<<grid, 128, 0, ctx->stream>>>(ctx->d_blob);
        CUF(cudaGetLastError());
    }
    CUF(cudaStreamSynchronize(ctx->stream));           // `blob` is pageable host memory
    // both kernels stage the static tables in dynamic shared memory; the create-time limit is 96 KB
    CUF(cudaFuncSetAttribute(simulate_mixed_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (96 + 64) * 1024));
    CUF(cudaFuncSetAttribute(simulate_mixed_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (96 + 64) * 1024));
    CUF(cudaFuncSetAttribute(finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (96 + 8) * 1024));
    CUF(cudaFuncSetAttribute(plan_mixed_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (96 + 24) * 1024));
    CUF(cudaFuncSetAttribute(plan_mixed_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (96 + 24) * 1024));
    CUF(cudaFuncSetAttribute(mixed_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (96 + 24) * 1024));
#undef CUF
    *out = ctx;
    return SAILOR_OK;
}

int sailor_destroy(sailor_ctx* ctx) {
    if (!ctx) return SAILOR_OK;
    DeviceGuard guard(ctx->device);
    if (ctx->d_blob) cudaStreamSynchronize(ctx->stream);
    cudaFree(ctx->d_blob);
    cudaFree(ctx->d_avail);
    cudaFreeHost(ctx->h_avail);
    cudaFree(ctx->d_ctrl);
    cudaFree(ctx->d_sim_error);
    cudaFreeHost(ctx->h_out);
    cudaFree(ctx->d_partial);
    cudaFree(ctx->d_partial_n);
    cudaFree(ctx->space.d_chunk_start);
    cudaFree(ctx->space.d_flat_base);
    cudaFree(ctx->space.d_live_start);
    cudaFree(ctx->space.d_cfg_closed);
    cudaFree(ctx->space.d_wave_start);
    cudaFree(ctx->space.d_cfg_best);
    cudaFree(ctx->space.d_groups);
    cudaFree(ctx->space.d_cfg_cache);
    cudaFree(ctx->d_stage);
    cudaFree(ctx->d_mix);
    cudaFree(ctx->d_dp);
    for (cudaEvent_t e : {ctx->ev0, ctx->ev1, ctx->ev2, ctx->evh0, ctx->evh1, ctx->ev_chunk, ctx->ev_join, ctx->ev_slot[0],
                          ctx->ev_slot[1], ctx->ev_slot[2]})
        if (e) cudaEventDestroy(e);
    if (ctx->out_stream) cudaStreamDestroy(ctx->out_stream);
    delete ctx;
    return SAILOR_OK;
}

int sailor_set_availability(sailor_ctx* ctx, const uint16_t* avail) {
    if (!ctx || !avail) return SAILOR_E_ARG;
    DeviceGuard guard(ctx->device);
    // A search takes the snapshot along in its launch parameters; the device copy that the other kernels read
    // through a pointer is brought up to date when one of them is next enqueued (upload_availability).  The pinned
    // buffer may still feed such a copy, unless the stream has been synchronised since.
    if (ctx->avail_epoch == ctx->sync_epoch) CU(ctx, stream_sync(ctx));
    memcpy(ctx->h_avail, avail, ctx->hdr.R * sizeof(uint16_t));
    ctx->avail_dirty = true;
    return SAILOR_OK;
}

int sailor_simulate(sailor_ctx* ctx, const sailor_plan_rec* plans, uint64_t n, int on_device, double* t_iter,
                    uint64_t* peak_mem, double* cost, uint32_t* status) {
    if (!ctx || (!plans && n)) return SAILOR_E_ARG;
    if (n == 0) return SAILOR_OK;
    if ((uintptr_t)plans % 8 != 0) return SAILOR_E_ARG;
    DeviceGuard guard(ctx->device);
    auto launch = [ctx](const sailor_plan_rec* d_plans, uint64_t m, double* d_t, uint64_t* d_m, double* d_c, uint32_t* d_s,
                        unsigned int* bad_flag) {
        const uint64_t tiles = (m + BATCH_POOL - 1) / BATCH_POOL;
        const uint64_t cap = (uint64_t)ctx->sm_count * BATCH_BLOCKS_PER_SM * 4;   // the resident blocks, four pools each at least
        const uint32_t grid = (uint32_t)(tiles < cap ? tiles : cap);
        simulate_kernel<<<grid, BATCH_THREADS, 0, ctx->stream>>>(ctx->d_blob, ctx->d_avail, d_plans, m, d_t, d_m, d_c, d_s, bad_flag);
        CU(ctx, cudaGetLastError());
        return (int)SAILOR_OK;
    };
    if (!on_device)                                               // records are checked by the kernel (SIM_ERR_BAD_RECORD)
        return host_batch(ctx, reinterpret_cast<const unsigned char*>(plans), sizeof(sailor_plan_rec), n, t_iter, peak_mem, cost,
                          status, [&](const unsigned char* d_recs, uint64_t m, double* d_t, uint64_t* d_m, double* d_c, uint32_t* d_s) {
                              return launch(reinterpret_cast<const sailor_plan_rec*>(d_recs), m, d_t, d_m, d_c, d_s, ctx->d_sim_error);
                          });
    {
        const int rc_up = upload_availability(ctx);
        if (rc_up) return rc_up;
    }
    return launch(plans, n, t_iter, peak_mem, cost, status, nullptr);
}

int sailor_simulate_mixed(sailor_ctx* ctx, const sailor_mixed_plan* plans, uint64_t n, int on_device, double* t_iter,
                          uint64_t* peak_mem, double* cost, uint32_t* status) {
    return sailor_simulate_mixed_strided(ctx, plans, n, (uint32_t)sizeof(sailor_mixed_plan), on_device, t_iter, peak_mem,
                                         cost, status);
}

int sailor_simulate_mixed_strided(sailor_ctx* ctx, const void* plans_v, uint64_t n, uint32_t record_bytes, int on_device,
                                  double* t_iter, uint64_t* peak_mem, double* cost, uint32_t* status) {
    constexpr uint32_t HEAD = (uint32_t)offsetof(sailor_mixed_plan, stage);
    if (!ctx || (!plans_v && n)) return SAILOR_E_ARG;
    if (record_bytes % 8 != 0 || record_bytes < HEAD + sizeof(sailor_mixed_stage) || record_bytes > sizeof(sailor_mixed_plan))
        return SAILOR_E_ARG;
    if (n == 0) return SAILOR_OK;
    const unsigned char* plans = static_cast<const unsigned char*>(plans_v);
    if ((uintptr_t)plans % 8 != 0) return SAILOR_E_ARG;
    const uint32_t max_stages = (record_bytes - HEAD) / (uint32_t)sizeof(sailor_mixed_stage);
    DeviceGuard guard(ctx->device);
    auto launch = [ctx, record_bytes, max_stages](const unsigned char* d_plans, uint64_t m, double* d_t, uint64_t* d_m, double* d_c,
                                                  uint32_t* d_s, uint32_t report_bad) {
        const uint64_t tiles = (m + SIM_THREADS / 32 - 1) / (SIM_THREADS / 32);     // a warp per plan
        const uint64_t cap = (uint64_t)ctx->sm_count * 32;
        const uint32_t grid = (uint32_t)(tiles < cap ? tiles : cap);
        const size_t smem = ctx->hdr.static_bytes + sizeof(unsigned long long) * (SIM_THREADS / 32) * ctx->hdr.R;
        unsigned int* deep_seen = ctx->d_sim_error + 1;
        if (max_stages > 32) CU(ctx, cudaMemsetAsync(deep_seen, 0, sizeof(unsigned int), ctx->stream));
        simulate_mixed_kernel<false><<<grid, SIM_THREADS, smem, ctx->stream>>>(ctx->d_blob, ctx->d_avail, d_plans, record_bytes,
                                                                                max_stages, m, d_t, d_m, d_c, d_s, ctx->d_sim_error,
                                                                                deep_seen, report_bad);
        CU(ctx, cudaGetLastError());
        if (max_stages > 32) {                                   // the plans of more than 32 stages, if the first launch saw any
            const uint64_t cap2 = (uint64_t)ctx->sm_count * 16;
            simulate_mixed_kernel<true><<<(uint32_t)(tiles < cap2 ? tiles : cap2), SIM_THREADS, smem, ctx->stream>>>(
                ctx->d_blob, ctx->d_avail, d_plans, record_bytes, max_stages, m, d_t, d_m, d_c, d_s, ctx->d_sim_error, deep_seen,
                report_bad);
            CU(ctx, cudaGetLastError());
        }
        return (int)SAILOR_OK;
    };
    if (!on_device)                                               // records are checked by the kernel (SIM_ERR_BAD_RECORD)
        return host_batch(ctx, plans, record_bytes, n, t_iter, peak_mem, cost, status,
                          [&](const unsigned char* d_recs, uint64_t m, double* d_t, uint64_t* d_m, double* d_c, uint32_t* d_s) {
                              return launch(d_recs, m, d_t, d_m, d_c, d_s, 1u);
                          });
    {
        const int rc_up = upload_availability(ctx);
        if (rc_up) return rc_up;
    }
    return launch(plans, n, t_iter, peak_mem, cost, status, 0u);
}

int sailor_space_size(const sailor_ctx* ctx, const sailor_space* s, uint64_t* n_out) {
    if (!n_out) return SAILOR_E_ARG;
    int rc = check_space(ctx, s);
    if (rc) return rc;
    return space_total(ctx, to_desc(s), n_out);
}

int sailor_decode(const sailor_ctx* ctx, const sailor_space* s, uint64_t flat, sailor_plan_rec* out) {
    if (!out) return SAILOR_E_ARG;
    int rc = check_space(ctx, s);
    if (rc) return rc;
    return decode_flat(to_desc(s), ctx->hdr.T, ctx->hdr.Z, flat, out) ? SAILOR_OK : SAILOR_E_RANGE;
}

static int plan_range_impl(sailor_ctx* ctx, const sailor_space* s, const sailor_objective* o, uint64_t flat_lo,
                           uint64_t flat_hi, uint32_t k, sailor_result* topk, uint32_t* n_found, sailor_stats* stats) {
    if (!ctx || !s || !o || !topk || !n_found || k == 0) return SAILOR_E_ARG;
    if (k > SAILOR_K_MAX || o->kind > SAILOR_OBJ_MAX_THROUGHPUT_PER_USD) return SAILOR_E_RANGE;
    if (std::isnan(o->budget_usd_per_iter) || std::isnan(o->min_iters_per_s) ||
        std::isnan(o->budget_factor_over_cheapest))
        return SAILOR_E_ARG;
    if (o->flags & ~(SAILOR_FLAG_EVAL_ALL | SAILOR_FLAG_DEGREE_ORDER | SAILOR_FLAG_MIN_TP_ONLY | SAILOR_FLAG_F32_SCREEN))
        return SAILOR_E_ARG;
    if ((o->flags & SAILOR_FLAG_F32_SCREEN) &&
        (o->budget_usd_per_iter > 0.0 || o->min_iters_per_s > 0.0 || o->budget_factor_over_cheapest > 0.0 ||
         (o->flags & SAILOR_FLAG_DEGREE_ORDER)))
        return SAILOR_E_ARG;                                   // the screen covers unconstrained searches
    DeviceGuard guard(ctx->device);
    int rc = prepare_space(ctx, s);
    if (rc) return rc;
    const uint64_t total = ctx->space.n_total;
    if (flat_hi > total) flat_hi = total;
    if (flat_lo > flat_hi) flat_lo = flat_hi;
    const bool waves = (o->flags & SAILOR_FLAG_DEGREE_ORDER) != 0;
    if (waves) {
        if (o->kind == SAILOR_OBJ_MAX_THROUGHPUT_PER_USD || (o->flags & SAILOR_FLAG_EVAL_ALL) || flat_lo != 0 ||
            flat_hi != total)
            return SAILOR_E_ARG;
        if (!ctx->space.d_cfg_closed) return SAILOR_E_RANGE;     // more configurations than the wave tables hold
    }

    uint32_t launches = 0;
    if (ctx->ctrl_dirty) {             // first search of the context, or the last one failed half-way
        CU(ctx, cudaMemsetAsync(ctx->d_ctrl, 0, sizeof(Ctrl), ctx->stream));
        CU(ctx, cudaMemsetAsync(&ctx->d_ctrl->min_cost_bits, 0x7f, 2 * sizeof(unsigned long long), ctx->stream));
    }
    ctx->ctrl_dirty = true;            // until this call has gone through
    if (stats) CU(ctx, cudaEventRecord(ctx->ev0, ctx->stream));
    const bool two_pass = o->budget_factor_over_cheapest > 0.0;
    // a whole-space search with pruning on walks only the prefixes the survey found live
    const bool live = !(o->flags & SAILOR_FLAG_EVAL_ALL) && flat_lo == 0 && flat_hi == total;
    bool launched = false;
    if (two_pass) {
        // cheapest feasible plan first; the block that ends that pass leaves factor * cost in ctrl->budget
        rc = enqueue_pass(ctx, SAILOR_OBJ_MIN_COST, 0.0, false, 0.0, o->flags, flat_lo, flat_hi, live, 1,
                          o->budget_factor_over_cheapest, &launches, &launched);
        if (rc) return rc;
    }
    rc = enqueue_pass(ctx, o->kind, o->budget_usd_per_iter, two_pass, o->min_iters_per_s, o->flags, flat_lo,
                      flat_hi, live, k, 0.0, &launches, &launched);
    if (rc) return rc;
    if (stats) CU(ctx, cudaEventRecord(ctx->ev1, ctx->stream));
    if (!launched) memset(&ctx->h_out->ctrl, 0, sizeof(Ctrl));    // an empty range: nothing ran, nothing was found
    CU(ctx, stream_sync(ctx));                                      // the results are in h_out once the kernels are done
    ctx->ctrl_dirty = false;
    const Ctrl& cr = ctx->h_out->ctrl;
    if (cr.error) return SAILOR_E_DEVICE;
    if (cr.n_found > k) return SAILOR_E_DEVICE;               // cannot happen; never copy past the caller's k records
    *n_found = cr.n_found;
    memcpy(topk, ctx->h_out->results, sizeof(sailor_result) * cr.n_found);
    if (stats) {
        // in live mode the kernels count the evaluated candidates only; the rest is the survey's closed form
        // (in degree order: of the configurations the waves selected, summed on the device)
        const SpaceCache& sc = ctx->space;
        const bool closed_form = live && !waves;
        stats->n_total = closed_form ? sc.closed[0] : cr.stats[0];
        stats->n_invalid = closed_form ? sc.closed[1] : cr.stats[1];
        stats->n_oom = closed_form ? sc.closed[2] : cr.stats[2];
        stats->n_pruned_tp = cr.stats[6];
        stats->n_skipped = waves ? sc.closed[0] - cr.stats[0] : 0;
        stats->n_configs = sc.n_config;
        stats->n_configs_evaluated = waves ? cr.n_cfg_evaluated : sc.n_config;
        stats->n_over_avail = cr.stats[3];
        stats->n_over_constraint = cr.stats[4];
        stats->n_feasible = cr.stats[5];
        stats->budget_used = two_pass ? (launched ? cr.budget : 0.0) : o->budget_usd_per_iter;
        double mc;
        memcpy(&mc, &cr.min_cost_bits, sizeof(mc));
        stats->min_feasible_cost = cr.stats[5] ? mc : 0.0;
        float ms = 0.f;
        CU(ctx, cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
        stats->kernel_ms = ms;
        stats->n_launches = launches;
        stats->d2h_ms = 0.f;               // no copy of its own: the results were written in place
        if (ctx->h2d_fresh) {              // an upload for another entry point was enqueued before this search: complete by now
            CU(ctx, cudaEventElapsedTime(&ctx->h2d_ms, ctx->evh0, ctx->evh1));
            ctx->h2d_fresh = false;
        }
        stats->h2d_ms = ctx->h2d_ms;
    }
    return SAILOR_OK;
}

int sailor_plan(sailor_ctx* ctx, const sailor_space* s, const sailor_objective* o, uint32_t k,
                sailor_result* topk, uint32_t* n_found, sailor_stats* stats) {
    return sailor_plan_range(ctx, s, o, 0, ~0ull >> 1, k, topk, n_found, stats);
}

}  // extern "C"

// ---- search without device allocation ----------------------------------------------------------
//
// sailor_plan_range keeps its per-space index arrays in memory it allocates when a new space
// arrives.  The variant below takes every byte of working memory from one fixed array that is
// part of the library image instead, so it can serve callers that must not allocate.

namespace {

constexpr uint32_t NOALLOC_GRID_MAX = 1024;     // blocks whose partial lists fit the fixed scratch

struct NoAllocScratch {                         // layout of the fixed scratch array
    Ctrl ctrl;
    PlanOut out;
    uint32_t partial_n[NOALLOC_GRID_MAX];
    Hit partial[(size_t)NOALLOC_GRID_MAX * SAILOR_K_MAX];
    uint32_t cfg_chunk_start[SAILOR_NOALLOC_CONFIG_MAX + 1];
    uint64_t cfg_flat_base[SAILOR_NOALLOC_CONFIG_MAX];
};

// About 0.6 MB, held by every GPU that loads the library until the process exits.  In host code
// this name is only a handle for cudaGetSymbolAddress; it is never passed to a kernel.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];
static_assert(offsetof(NoAllocScratch, partial) % 16 == 0, "the lists are read 16 bytes at a time");

constexpr int NOALLOC_DEVICES_MAX = 64;
// device address of the array, per device (atomic: two threads resolving it together store the same address)
std::atomic<NoAllocScratch*> g_noalloc_ptr[NOALLOC_DEVICES_MAX];
// resident blocks per SM of each kernel variant at a given shared-memory size, per device (0 = not asked yet)
struct OccupancyMemo { std::atomic<uint64_t> smem_and_blocks; };
OccupancyMemo g_noalloc_occ[NOALLOC_DEVICES_MAX][PLAN_VARIANTS];

// Device address of the scratch on the current device; resolved on first use per device.
int noalloc_scratch(sailor_ctx* ctx, NoAllocScratch** out) {
    if (ctx->device < 0 || ctx->device >= NOALLOC_DEVICES_MAX) return SAILOR_E_RANGE;
    NoAllocScratch* known = g_noalloc_ptr[ctx->device].load(std::memory_order_acquire);
    if (!known) {
        void* p = nullptr;
        CU(ctx, cudaGetSymbolAddress(&p, g_noalloc_scratch));
        known = static_cast<NoAllocScratch*>(p);
        g_noalloc_ptr[ctx->device].store(known, std::memory_order_release);
    }
    *out = known;
    return SAILOR_OK;
}

// One pass (clear, search with its merge) whose scratch all lies in `sc`.
int enqueue_pass_noalloc(sailor_ctx* ctx, NoAllocScratch* sc, const SpaceDesc& desc, uint32_t n_config,
                         uint32_t p_max, size_t smem, uint32_t chunk_lo, uint32_t chunk_hi, uint64_t total,
                         uint32_t obj, double budget, bool budget_from_ctrl, double min_rate, uint32_t flags,
                         uint32_t k, double next_budget_factor, uint32_t* n_launches) {
    // the array keeps the previous call's contents: counters and the work counter restart at zero
    CU(ctx, cudaMemsetAsync(&sc->ctrl, 0, offsetof(Ctrl, min_cost_bits), ctx->stream));
    CU(ctx, cudaMemsetAsync(&sc->ctrl.min_cost_bits, 0x7f, 2 * sizeof(unsigned long long), ctx->stream));
    PlanParams pp;
    memset(&pp, 0, sizeof(pp));
    pp.blob = ctx->d_blob;
    memcpy(pp.avail, ctx->h_avail, sizeof(pp.avail));
    pp.cfg_chunk_start = sc->cfg_chunk_start;
    pp.cfg_flat_base = sc->cfg_flat_base;
    pp.ctrl = &sc->ctrl;
    pp.partial = sc->partial;
    pp.partial_n = sc->partial_n;
    pp.sp = desc;
    pp.n_config = n_config;
    pp.flat_lo = 0;
    pp.flat_hi = total;
    pp.k = k;
    pp.eval_all = (flags & SAILOR_FLAG_EVAL_ALL) ? 1u : 0u;
    pp.min_tp_only = (flags & SAILOR_FLAG_MIN_TP_ONLY) ? 1u : 0u;
    pp.budget_from_ctrl = budget_from_ctrl ? 1u : 0u;
    pp.p_max = p_max;
    pp.budget = budget;
    pp.min_rate = min_rate;
    pp.chunk_lo = chunk_lo;
    pp.chunk_hi = chunk_hi;
    pp.out = &sc->out;
    pp.finish = 1;
    pp.next_budget_factor = next_budget_factor;
    pp.cost_only = next_budget_factor > 0.0 ? 1u : 0u;
    const uint32_t n_chunks = chunk_hi - chunk_lo;
    const bool constr = budget_from_ctrl || budget > 0.0 || min_rate > 0.0;
    PlanKernel kern = pick_kernel(obj, constr, true);
    const uint32_t variant = variant_of(obj, constr, true);
    {
        const int rc_opt = smem_optin(ctx, kern, variant);
        if (rc_opt) return rc_opt;
    }
    // the occupancy query costs host time on a path that exists for its latency: ask once per (device, variant, size)
    int per_sm = 0;
    std::atomic<uint64_t>& memo = g_noalloc_occ[ctx->device][variant].smem_and_blocks;
    const uint64_t seen = memo.load(std::memory_order_acquire);
    if (seen && (seen >> 8) == (uint64_t)smem) per_sm = (int)(seen & 0xff);
    else {
        CU(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, PLAN_THREADS, smem));
        if (per_sm >= 1 && per_sm < 256) memo.store(((uint64_t)smem << 8) | (uint64_t)per_sm, std::memory_order_release);
    }
    if (per_sm < 1) return SAILOR_E_RANGE;
    uint32_t grid = (uint32_t)per_sm * (uint32_t)ctx->sm_count;
    if (grid > NOALLOC_GRID_MAX) grid = NOALLOC_GRID_MAX;
    if (grid > n_chunks) grid = n_chunks;
    const uint32_t batch = n_chunks / (grid * 32u);
    pp.batch = batch < 1 ? 1 : (batch > 16 ? 16 : batch);
    kern<<<grid, PLAN_THREADS, smem, ctx->stream>>>(pp);
    CU(ctx, cudaGetLastError());
    ++*n_launches;
    return SAILOR_OK;
}

}  // namespace

extern "C" int sailor_plan_noalloc(sailor_ctx* ctx, const sailor_space* s, const sailor_objective* o, uint32_t k,
                                   sailor_result* topk, uint32_t* n_found, sailor_stats* stats) {
    if (!ctx || !s || !o || !topk || !n_found || k == 0) return SAILOR_E_ARG;
    if (k > SAILOR_K_MAX || o->kind > SAILOR_OBJ_MAX_THROUGHPUT_PER_USD) return SAILOR_E_RANGE;
    if (std::isnan(o->budget_usd_per_iter) || std::isnan(o->min_iters_per_s) ||
        std::isnan(o->budget_factor_over_cheapest))
        return SAILOR_E_ARG;
    if (o->flags & ~(SAILOR_FLAG_EVAL_ALL | SAILOR_FLAG_MIN_TP_ONLY)) return SAILOR_E_ARG;   // degree order needs tables this variant has no room for
    int rc = check_space(ctx, s);
    if (rc) return rc;
    const SpaceDesc d = to_desc(s);
    uint64_t total = 0;
    rc = space_total(ctx, d, &total);
    if (rc) return rc;
    const uint32_t per_p = d.n_mbs * d.n_tp * d.n_rc * d.n_d;
    const uint64_t n_config = (uint64_t)per_p * d.n_p;
    if (n_config > SAILOR_NOALLOC_CONFIG_MAX) return SAILOR_E_RANGE;       // beyond the fixed scratch

    // per-configuration offsets, built in fixed-size host arrays (thread-local: no heap, no device memory)
    static thread_local uint32_t h_chunk_start[SAILOR_NOALLOC_CONFIG_MAX + 1];
    static thread_local uint64_t h_flat_base[SAILOR_NOALLOC_CONFIG_MAX];
    const uint64_t R = ctx->hdr.R;
    uint64_t chunks = 0, flat = 0;
    uint32_t p_max = 0;
    for (uint32_t j = 0; j < d.n_p; ++j) {
        const uint32_t nseg = nseg_of(d.p_values[j], d.seg_max);
        p_max = d.p_values[j] > p_max ? d.p_values[j] : p_max;
        const uint64_t items = ipow64(R, nseg - 1);
        const uint64_t per_cfg = (items + PLAN_THREADS - 1) / PLAN_THREADS;
        for (uint32_t c = 0; c < per_p; ++c) {
            h_chunk_start[(size_t)j * per_p + c] = (uint32_t)chunks;
            h_flat_base[(size_t)j * per_p + c] = flat;
            chunks += per_cfg;
            flat += items * R;
            if (chunks >= 0xfff00000ull) return SAILOR_E_RANGE;
        }
    }
    h_chunk_start[n_config] = (uint32_t)chunks;
    const size_t smem = plan_smem_bytes(ctx->hdr.static_bytes, p_max, ctx->hdr.T, ctx->hdr.Z, (uint32_t)n_config);
    if (smem > 200 * 1024) return SAILOR_E_RANGE;

    DeviceGuard guard(ctx->device);
    NoAllocScratch* sc = nullptr;
    rc = noalloc_scratch(ctx, &sc);
    if (rc) return rc;
    // the host arrays are reused by the next call on this thread: once a copy from them is enqueued, no path
    // leaves this function without waiting for the stream
    cudaError_t ce = cudaMemcpyAsync(sc->cfg_chunk_start, h_chunk_start, (n_config + 1) * sizeof(uint32_t),
                                     cudaMemcpyHostToDevice, ctx->stream);
    if (ce == cudaSuccess)
        ce = cudaMemcpyAsync(sc->cfg_flat_base, h_flat_base, n_config * sizeof(uint64_t), cudaMemcpyHostToDevice, ctx->stream);
    if (ce == cudaSuccess) ce = cudaMemsetAsync(&sc->ctrl, 0, sizeof(Ctrl), ctx->stream);      // also the error word
    if (ce == cudaSuccess) ce = cudaMemsetAsync(&sc->out.ctrl, 0, sizeof(Ctrl), ctx->stream);  // read back even if nothing runs

    uint32_t launches = 0;
    if (ce == cudaSuccess) ce = cudaEventRecord(ctx->ev0, ctx->stream);
    const bool two_pass = o->budget_factor_over_cheapest > 0.0;
    rc = SAILOR_OK;
    if (ce == cudaSuccess && total > 0) {
        if (two_pass)
            rc = enqueue_pass_noalloc(ctx, sc, d, (uint32_t)n_config, p_max, smem, 0, (uint32_t)chunks, total,
                                      SAILOR_OBJ_MIN_COST, 0.0, false, 0.0, o->flags, 1,
                                      o->budget_factor_over_cheapest, &launches);
        if (rc == SAILOR_OK)
            rc = enqueue_pass_noalloc(ctx, sc, d, (uint32_t)n_config, p_max, smem, 0, (uint32_t)chunks, total, o->kind,
                                      o->budget_usd_per_iter, two_pass, o->min_iters_per_s, o->flags, k, 0.0, &launches);
    }
    if (ce == cudaSuccess && rc == SAILOR_OK) ce = cudaEventRecord(ctx->ev1, ctx->stream);
    if (ce == cudaSuccess && rc == SAILOR_OK)
        ce = cudaMemcpyAsync(ctx->h_out, &sc->out, sizeof(Ctrl) + sizeof(sailor_result) * k, cudaMemcpyDeviceToHost, ctx->stream);
    if (ce == cudaSuccess && rc == SAILOR_OK && stats) ce = cudaEventRecord(ctx->ev2, ctx->stream);
    {
        const cudaError_t se = stream_sync(ctx);               // on every path: the copies above read this thread's arrays
        if (ce == cudaSuccess) ce = se;
    }
    if (ce != cudaSuccess) { ctx->last_cuda = (int)ce; return SAILOR_E_CUDA; }
    if (rc) return rc;
    const Ctrl& cr = ctx->h_out->ctrl;
    if (cr.error) return SAILOR_E_DEVICE;
    // overlapping calls race on the shared array (documented): whatever they left, never copy past k records
    if (cr.n_found > k) return SAILOR_E_DEVICE;
    *n_found = cr.n_found;
    memcpy(topk, ctx->h_out->results, sizeof(sailor_result) * cr.n_found);
    if (stats) {
        stats->n_total = cr.stats[0];
        stats->n_invalid = cr.stats[1];
        stats->n_oom = cr.stats[2];
        stats->n_over_avail = cr.stats[3];
        stats->n_over_constraint = cr.stats[4];
        stats->n_feasible = cr.stats[5];
        stats->n_pruned_tp = cr.stats[6];
        stats->n_skipped = 0;
        stats->n_configs = stats->n_configs_evaluated = (uint32_t)n_config;
        stats->budget_used = two_pass ? cr.budget : o->budget_usd_per_iter;
        double mc;
        memcpy(&mc, &cr.min_cost_bits, sizeof(mc));
        stats->min_feasible_cost = cr.stats[5] ? mc : 0.0;
        float ms = 0.f;
        CU(ctx, cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
        stats->kernel_ms = ms;
        stats->n_launches = launches;
        stats->d2h_ms = 0.f;
        CU(ctx, cudaEventElapsedTime(&stats->d2h_ms, ctx->ev1, ctx->ev2));
        if (ctx->h2d_fresh) {
            CU(ctx, cudaEventElapsedTime(&ctx->h2d_ms, ctx->evh0, ctx->evh1));
            ctx->h2d_fresh = false;
        }
        stats->h2d_ms = ctx->h2d_ms;
    }
    return SAILOR_OK;
}

// ---- per-stage GPU types by dynamic programming ---------------------------------------------------

namespace {

struct Bump {                       // carves 256-byte aligned pieces out of one device buffer
    unsigned char* base;
    size_t at = 0;
    template <typename T>
    T* take(size_t n) {
        T* p = reinterpret_cast<T*>(base + at);
        at += (n * sizeof(T) + 255) & ~(size_t)255;
        return p;
    }
};

size_t padded(size_t bytes) { return (bytes + 255) & ~(size_t)255; }

}  // namespace

// The recursion steered by the budget (Sec. 4.2.3): one thread per problem, depth first.
static int plan_dp_budget_impl(sailor_ctx* ctx, const SpaceDesc& d, const sailor_zone_order* orders, uint32_t n_orders,
                               const sailor_objective* o, uint64_t workspace_bytes, uint32_t k, sailor_dp_result* topk,
                               uint32_t* n_found, sailor_dp_stats* stats) {
    const TabHdr& h = ctx->hdr;
    const uint32_t T = h.T;
    const uint64_t n_config = (uint64_t)d.n_p * d.n_mbs * d.n_tp * d.n_rc * d.n_d, n_problems = n_config * n_orders;
    uint32_t p_max = 0;
    for (uint32_t j = 0; j < d.n_p; ++j) p_max = d.p_values[j] > p_max ? d.p_values[j] : p_max;
    // what first fit needs of every problem, from the availability last set (host copy)
    std::vector<DpProblem> prob(n_problems);
    for (uint64_t c = 0; c < n_config; ++c) {
        const Config cf = config_of(d, (uint32_t)c);
        const uint64_t need = (uint64_t)cf.D * h.tp_values[cf.tpi];
        for (uint32_t q = 0; q < n_orders; ++q) {
            DpProblem& pb = prob[c * n_orders + q];
            memset(&pb, 0, sizeof(pb));
            pb.config = (uint32_t)c; pb.order = q; pb.index = (uint32_t)(c * n_orders + q);
            pb.P = cf.P; pb.nz = orders[q].n; pb.need = (uint32_t)(need > 0xffffffffull ? 0xffffffffull : need);
            memset(pb.first_later, DP_NONE, sizeof(pb.first_later));
            for (uint32_t zp = 0; zp < pb.nz; ++zp) {
                pb.zone[zp] = orders[q].zone[zp];
                for (uint32_t g = 0; g < T; ++g) {
                    const uint64_t cap = ctx->h_avail[pb.zone[zp] * T + g] / need;
                    pb.cap[zp][g] = (uint8_t)(cap > 255 ? 255 : cap);
                }
            }
            for (uint32_t zp = 0; zp < pb.nz; ++zp)
                for (uint32_t g = 0; g < T; ++g)
                    for (uint32_t later = zp + 1; later < pb.nz; ++later)
                        if (pb.cap[later][g] >= 1) { pb.first_later[zp][g] = (uint8_t)later; break; }
        }
    }
    DeviceGuard guard(ctx->device);
    DpTabLayout lay;
    lay.p_max = p_max; lay.T = T; lay.R = h.R;
    const size_t tab_bytes = (size_t)n_config * lay.stride() * sizeof(double);
    const size_t total = padded(tab_bytes) + padded(n_problems * sizeof(DpResult)) + padded(n_problems * sizeof(DpProblem)) +
                         padded(n_problems * DP_BUDGET_P_MAX * sizeof(DpbFrame)) + padded(sizeof(sailor_dp_result) * SAILOR_K_MAX) +
                         padded(40) + 4096;
    if (total > workspace_bytes) return SAILOR_E_RANGE;
    if (total > ctx->dp_bytes) {
        CU(ctx, stream_sync(ctx));
        cudaFree(ctx->d_dp);
        ctx->d_dp = nullptr;
        ctx->dp_bytes = 0;
        cudaError_t e = cudaMalloc(&ctx->d_dp, total);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SAILOR_E_NOMEM; }
        ctx->dp_bytes = total;
    }
    Bump bump{ctx->d_dp};
    double* d_tabs = bump.take<double>(tab_bytes / sizeof(double));
    DpResult* d_results = bump.take<DpResult>(n_problems);
    DpProblem* d_problems = bump.take<DpProblem>(n_problems);
    DpbFrame* d_frames = bump.take<DpbFrame>(n_problems * DP_BUDGET_P_MAX);
    sailor_dp_result* d_out = bump.take<sailor_dp_result>(SAILOR_K_MAX);
    unsigned long long* d_counters = bump.take<unsigned long long>(5);

    uint32_t launches = 0;
    {
        const int rc_up = upload_availability(ctx);
        if (rc_up) return rc_up;
    }
    CU(ctx, cudaEventRecord(ctx->ev0, ctx->stream));
    CU(ctx, cudaMemsetAsync(d_tabs, 0, tab_bytes, ctx->stream));
    CU(ctx, cudaMemsetAsync(d_counters, 0, 40, ctx->stream));
    CU(ctx, cudaMemcpyAsync(d_problems, prob.data(), n_problems * sizeof(DpProblem), cudaMemcpyHostToDevice, ctx->stream));
    {
        const uint32_t grid = (uint32_t)(n_config < 4096 ? n_config : 4096);
        dp_tables_kernel<<<grid, DP_THREADS, 0, ctx->stream>>>(ctx->d_blob, d, (uint32_t)n_config, lay, d_tabs);
        CU(ctx, cudaGetLastError());
        ++launches;
    }
    DpBudgetParams bp;
    memset(&bp, 0, sizeof(bp));
    bp.blob = ctx->d_blob; bp.avail = ctx->d_avail; bp.sp = d; bp.problems = d_problems; bp.tabs = d_tabs;
    bp.results = d_results; bp.frames = d_frames; bp.counters = d_counters; bp.lay = lay;
    bp.n_problems = (uint32_t)n_problems; bp.T = T;
    bp.limit = o->budget_usd_per_iter;
    bp.node_limit = 1ull << 24;
    dp_budget_kernel<<<(uint32_t)((n_problems + 63) / 64), 64, 0, ctx->stream>>>(bp);
    CU(ctx, cudaGetLastError());
    ++launches;
    DpSelectParams sel;
    memset(&sel, 0, sizeof(sel));
    sel.results = d_results; sel.out = d_out; sel.counters = d_counters;
    sel.sp = d; sel.n_problems = (uint32_t)n_problems; sel.n_orders = n_orders; sel.k = k;
    sel.budget = o->budget_usd_per_iter; sel.min_rate = o->min_iters_per_s;
    dp_select_kernel<<<1, DP_SELECT_THREADS, 0, ctx->stream>>>(sel);
    CU(ctx, cudaGetLastError());
    ++launches;
    CU(ctx, cudaEventRecord(ctx->ev1, ctx->stream));
    unsigned long long counters[5] = {0, 0, 0, 0, 0};
    std::vector<sailor_dp_result> host_out(k);
    CU(ctx, cudaMemcpyAsync(counters, d_counters, sizeof(counters), cudaMemcpyDeviceToHost, ctx->stream));
    CU(ctx, cudaMemcpyAsync(host_out.data(), d_out, sizeof(sailor_dp_result) * k, cudaMemcpyDeviceToHost, ctx->stream));
    CU(ctx, stream_sync(ctx));                                 // also: `prob` is pageable
    if (counters[1] > k) return SAILOR_E_DEVICE;
    *n_found = (uint32_t)counters[1];
    memcpy(topk, host_out.data(), sizeof(sailor_dp_result) * counters[1]);
    if (stats) {
        stats->n_problems = n_problems;
        stats->n_solved = counters[0];
        stats->n_over_constraint = counters[2];
        stats->n_states = counters[4];
        stats->workspace_used = total;
        float ms = 0.f;
        CU(ctx, cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
        stats->kernel_ms = ms;
        stats->n_launches = launches;
        stats->n_batches = 1;
        stats->n_unfinished = (uint32_t)counters[3];
    }
    return SAILOR_OK;
}

static int plan_dp_impl(sailor_ctx* ctx, const sailor_space* s, const sailor_zone_order* orders,
                        uint32_t n_orders, const sailor_objective* o, uint64_t workspace_bytes, uint32_t k,
                        sailor_dp_result* topk, uint32_t* n_found, sailor_dp_stats* stats) {
    if (!ctx || !s || !orders || !o || !topk || !n_found || k == 0 || n_orders == 0) return SAILOR_E_ARG;
    if (k > SAILOR_K_MAX) return SAILOR_E_RANGE;
    // the recursion minimises iteration time; a constraint is checked on the plan it returns per problem
    constexpr uint32_t dp_flags = SAILOR_DP_FLAG_INDEX_DENSE | SAILOR_DP_FLAG_INDEX_COMPACT | SAILOR_DP_FLAG_ENUM_BY_TYPE |
                                  SAILOR_DP_FLAG_ENUM_BY_ENTRY | SAILOR_DP_FLAG_BUDGET_LOOP;
    if (o->kind != SAILOR_OBJ_MAX_THROUGHPUT || (o->flags & ~dp_flags) != 0 ||
        ((o->flags & SAILOR_DP_FLAG_INDEX_DENSE) && (o->flags & SAILOR_DP_FLAG_INDEX_COMPACT)) ||
        ((o->flags & SAILOR_DP_FLAG_ENUM_BY_TYPE) && (o->flags & SAILOR_DP_FLAG_ENUM_BY_ENTRY)) ||
        o->budget_factor_over_cheapest > 0.0 ||
        std::isnan(o->budget_usd_per_iter) || std::isnan(o->min_iters_per_s) || std::isnan(o->budget_factor_over_cheapest))
        return SAILOR_E_ARG;
    int rc = check_space(ctx, s);
    if (rc) return rc;
    const TabHdr& h = ctx->hdr;
    const uint32_t T = h.T, Z = h.Z;
    for (uint32_t q = 0; q < n_orders; ++q) {
        if (orders[q].n < 1 || orders[q].n > Z) return SAILOR_E_ARG;
        uint32_t seen = 0;
        for (uint32_t j = 0; j < orders[q].n; ++j) {
            if (orders[q].zone[j] >= Z || ((seen >> orders[q].zone[j]) & 1u)) return SAILOR_E_ARG;
            seen |= 1u << orders[q].zone[j];
        }
    }
    const SpaceDesc d = to_desc(s);
    const uint64_t n_config = (uint64_t)d.n_p * d.n_mbs * d.n_tp * d.n_rc * d.n_d;
    if (n_config * n_orders > (1u << 22)) return SAILOR_E_RANGE;
    if (workspace_bytes == 0) workspace_bytes = 8ull << 30;
    uint32_t p_max = 0;
    for (uint32_t j = 0; j < d.n_p; ++j) p_max = d.p_values[j] > p_max ? d.p_values[j] : p_max;
    if (o->flags & SAILOR_DP_FLAG_BUDGET_LOOP) {
        if (!(o->budget_usd_per_iter > 0.0)) return SAILOR_E_ARG;
        if (p_max > DP_BUDGET_P_MAX) return SAILOR_E_RANGE;
        return plan_dp_budget_impl(ctx, d, orders, n_orders, o, workspace_bytes, k, topk, n_found, stats);
    }

    // every problem's table layout, from the availability last set (host copy)
    const uint64_t n_problems = n_config * n_orders;
    std::vector<DpProblem> prob(n_problems);
    std::vector<uint32_t> vtabs;        // rank tables of the compactly indexed zone positions, all problems
    // how a zone position's count vectors are indexed: 0 = the smaller of the two ways, 1 = mixed radix whenever it
    // fits, 2 = by rank whenever it fits (SAILOR_DP_FLAG_INDEX_*)
    const int index_mode = (o->flags & SAILOR_DP_FLAG_INDEX_DENSE) ? 1 : (o->flags & SAILOR_DP_FLAG_INDEX_COMPACT) ? 2 : 0;
    // which threads a stage's launch has: one per count vector the stage can have reached ("live", whenever every
    // zone position has its rank table), or one per table entry (SAILOR_DP_FLAG_ENUM_BY_ENTRY)
    bool all_live = !(o->flags & SAILOR_DP_FLAG_ENUM_BY_ENTRY);
    std::vector<uint64_t> V, live_stage;                     // scratch of the loop below
    std::vector<uint64_t> live_off(n_problems + 1, 0);      // per problem: where its per-stage live counts start
    std::vector<uint32_t> live_cnt;                          // count vectors stage i can have reached, all positions
    uint64_t n_states = 0;
    uint32_t vt_len_max = 0;                                 // words of the largest problem's rank tables
    std::map<std::array<uint64_t, 3>, uint64_t> same_states;
    for (uint64_t c = 0; c < n_config; ++c) {
        const Config cf = config_of(d, (uint32_t)c);
        const uint32_t tp = h.tp_values[cf.tpi];
        const uint64_t dm = (uint64_t)cf.D * h.mbs_values[cf.mi];
        const bool valid = h.gbs % dm == 0 && h.heads % tp == 0;
        const uint64_t need = (uint64_t)cf.D * tp;
        for (uint32_t q = 0; q < n_orders; ++q) {
            DpProblem& pb = prob[c * n_orders + q];
            memset(&pb, 0, sizeof(pb));
            pb.config = (uint32_t)c; pb.order = q; pb.index = (uint32_t)(c * n_orders + q);
            pb.P = cf.P; pb.nz = orders[q].n; pb.need = (uint32_t)(need > 0xffffffffull ? 0xffffffffull : need);
            memset(pb.first_later, DP_NONE, sizeof(pb.first_later));
            live_off[c * n_orders + q] = live_cnt.size();
            if (!valid) continue;                           // no entries: the finish step finds no plan
            // the states, their index and the rank tables depend on (P, D * tp, zone order) only: configurations
            // that differ in the microbatch size or in recomputation take them from the first such problem
            const std::array<uint64_t, 3> key = {cf.P, need, q};
            const auto seen = same_states.find(key);
            if (seen != same_states.end()) {
                const DpProblem& first = prob[seen->second];
                const uint32_t config = pb.config, index = pb.index;
                pb = first;
                pb.config = config; pb.index = index;
                live_off[c * n_orders + q] = live_off[seen->second];
                n_states += (uint64_t)pb.n_lvl * cf.P;
                continue;
            }
            same_states.emplace(key, c * n_orders + q);
            uint64_t n_lvl = 0;
            pb.vt_lo = (uint32_t)vtabs.size();
            live_stage.assign(cf.P, 0);
            for (uint32_t zp = 0; zp < pb.nz; ++zp) {
                pb.zone[zp] = orders[q].zone[zp];
                // counted types: the zone can host some but not all P stages of them
                uint32_t counted[SAILOR_T_MAX], m = 0;
                uint64_t dense = 1;
                bool dense_ok = true;
                for (uint32_t g = 0; g < T; ++g) {
                    const uint64_t cap = ctx->h_avail[pb.zone[zp] * T + g] / need;
                    pb.cap[zp][g] = (uint8_t)(cap > 255 ? 255 : cap);
                    if (cap >= 1 && cap < cf.P) {
                        counted[m++] = g;
                        if (dense_ok) dense *= cap + 1;
                        if (dense > (1ull << 31)) dense_ok = false;
                    }
                }
                pb.n_counted[zp] = (uint8_t)m;
                // compact index: count vectors within the caps that add up to at most P (rank tables V[j][s])
                const uint32_t w = cf.P + 1;
                V.assign((size_t)(m + 1) * w, 0);
                for (uint32_t sgm = 0; sgm < w; ++sgm) V[(size_t)m * w + sgm] = sgm + 1;           // W = 1 each
                bool compact_ok = true;
                for (uint32_t j = m; j-- > 0;) {
                    const uint64_t cj = pb.cap[zp][counted[j]];
                    uint64_t run = 0;
                    for (uint32_t sgm = 0; sgm < w; ++sgm) {
                        const uint64_t lo = sgm > cj ? V[(size_t)(j + 1) * w + (sgm - cj - 1)] : 0;
                        run += V[(size_t)(j + 1) * w + sgm] - lo;                                  // W[j][s]
                        V[(size_t)j * w + sgm] = run;
                        if (run > (1ull << 31)) compact_ok = false;
                    }
                }
                const uint64_t compact = m ? V[cf.P] - (cf.P ? V[cf.P - 1] : 0) : 1;                // W[0][P]
                if (!dense_ok && !compact_ok) return SAILOR_E_RANGE;
                const bool use_compact = index_mode == 2 ? compact_ok && m > 0
                                         : index_mode == 1 ? !dense_ok
                                                           : (m > 0 && compact_ok && (!dense_ok || dense > 4 * compact));
                uint64_t S = 1;
                pb.rank_off[zp] = DP_DENSE;
                if (m > 0 && compact_ok) {                   // the rank table serves the live enumeration in any case
                    pb.rank_off[zp] = (uint32_t)vtabs.size();
                    for (uint64_t x : V) vtabs.push_back((uint32_t)x);
                    if (vtabs.size() > (1ull << 30)) return SAILOR_E_RANGE;
                } else if (m > 0) {
                    all_live = false;
                }
                for (uint32_t st = 0; st < cf.P; ++st) {     // count vectors with at most st + 1 stages
                    const uint32_t bud = st + 1;
                    live_stage[st] += m > 0 && compact_ok ? V[bud] - V[bud - 1] : 1;
                }
                if (use_compact) {
                    S = compact;
                    pb.vt_off[zp] = pb.rank_off[zp];
                    for (uint32_t j = 0; j < m; ++j) {
                        // rank of "one stage of type counted[j]": every vector that has a zero there and is zero before it
                        // comes first: V[j+1][P] - V[j+1][P-1] ... summed by the rank formula with u = e_j
                        pb.stride[zp][counted[j]] = 1;                                         // marks the type as counted
                        pb.first_idx[zp][counted[j]] = (uint32_t)(V[(size_t)(j + 1) * w + cf.P] - V[(size_t)(j + 1) * w + cf.P - 1]);
                    }
                } else {
                    pb.vt_off[zp] = DP_DENSE;
                    for (uint32_t j = 0; j < m; ++j) {
                        const uint32_t g = counted[j];
                        pb.magic[zp][g] = ~0ull / (pb.cap[zp][g] + 1ull) + 1;                  // ceil(2^64 / (cap + 1)), cap + 1 >= 2
                        pb.stride[zp][g] = (uint32_t)S;
                        pb.first_idx[zp][g] = (uint32_t)S;
                        S *= pb.cap[zp][g] + 1ull;
                    }
                }
                pb.S[zp] = (uint32_t)S;
                pb.zp_base[zp] = (uint32_t)n_lvl;
                n_lvl += (uint64_t)T * S;
                if (n_lvl > (1ull << 31)) return SAILOR_E_RANGE;
            }
            pb.zp_base[pb.nz] = (uint32_t)n_lvl;
            for (uint32_t zp = 0; zp < pb.nz; ++zp)
                for (uint32_t g = 0; g < T; ++g)
                    for (uint32_t q = zp + 1; q < pb.nz; ++q)
                        if (pb.cap[q][g] >= 1) { pb.first_later[zp][g] = (uint8_t)q; break; }
            pb.n_lvl = (uint32_t)n_lvl;
            pb.vt_len = (uint32_t)(vtabs.size() - pb.vt_lo);
            vt_len_max = pb.vt_len > vt_len_max ? pb.vt_len : vt_len_max;
            n_states += n_lvl * cf.P;
            for (uint32_t st = 0; st < cf.P; ++st) live_cnt.push_back((uint32_t)(live_stage[st] > n_lvl ? n_lvl : live_stage[st]));   // <= n_lvl / T
        }
    }
    // deepest pipelines first, so that the launch for a distance from the last stage covers a prefix
    std::vector<uint32_t> by_depth;
    by_depth.reserve(n_problems);
    for (uint64_t j = 0; j < n_problems; ++j)
        if (prob[j].n_lvl) by_depth.push_back((uint32_t)j);
    std::stable_sort(by_depth.begin(), by_depth.end(), [&](uint32_t a, uint32_t b) { return prob[a].P > prob[b].P; });
    auto work_bytes = [](const DpProblem& pb) { return (uint64_t)pb.n_lvl * (2 * sizeof(DpVal) + pb.P); };
    struct Batch { size_t first, count; uint64_t entries, choice_bytes, blocks; };
    std::vector<Batch> batches;
    uint64_t largest = 0;
    for (size_t j = 0; j < by_depth.size();) {
        Batch b = {j, 0, 0, 0, 0};
        uint64_t bytes = 0;
        while (j < by_depth.size()) {
            const DpProblem& pb = prob[by_depth[j]];
            const uint64_t wb = work_bytes(pb) + 512;
            if (b.count && bytes + wb > workspace_bytes) break;
            if (wb > workspace_bytes) return SAILOR_E_RANGE;      // one problem alone does not fit
            bytes += wb;
            b.entries += pb.n_lvl;
            b.choice_bytes += (uint64_t)pb.n_lvl * pb.P;
            b.blocks += all_live ? (uint64_t)pb.P + 1 : (pb.n_lvl + DP_THREADS - 1) / DP_THREADS;   // words of the block lists
            ++b.count; ++j;
        }
        largest = bytes > largest ? bytes : largest;
        batches.push_back(b);
    }
    uint64_t max_entries = 0, max_choice = 0, max_blocks = 0, max_count = 0;
    for (const Batch& b : batches) {
        max_entries = std::max(max_entries, b.entries);
        max_choice = std::max(max_choice, b.choice_bytes);
        max_blocks = std::max(max_blocks, b.blocks);
        max_count = std::max<uint64_t>(max_count, b.count);
    }
    if (max_blocks > 0x7fffffffull) return SAILOR_E_RANGE;
    if (all_live) {                                        // what the launches visit: live count vectors only
        n_states = 0;
        for (uint64_t j = 0; j < n_problems; ++j)
            for (uint32_t st = 0; prob[j].n_lvl && st < prob[j].P; ++st) n_states += (uint64_t)live_cnt[live_off[j] + st] * T;
    }
    // a thread per count vector for all its types at once, or a thread per (count vector, type)
    // (its blocks stage their problem's rank tables in shared memory: at most Z * (T + 1) * (P + 1) words)
    const bool by_vector = all_live && vt_len_max * 4 <= 40 * 1024 && !(o->flags & SAILOR_DP_FLAG_ENUM_BY_TYPE);
    const uint32_t live_mult = by_vector ? 1u : T;

    DeviceGuard guard(ctx->device);
    DpTabLayout lay;
    lay.p_max = p_max; lay.T = T; lay.R = h.R;
    const size_t tab_bytes = (size_t)n_config * lay.stride() * sizeof(double);
    const size_t total = padded(tab_bytes) + padded(vtabs.size() * sizeof(uint32_t) + 4) + padded(n_problems * sizeof(DpResult)) +
                         padded(n_problems * sizeof(DpProblem)) +
                         2 * padded((max_blocks + p_max + 16) * sizeof(uint32_t)) + 2 * padded(max_entries * sizeof(DpVal)) +
                         padded(max_choice) + padded(sizeof(sailor_dp_result) * SAILOR_K_MAX) + padded(24) + 4096;
    if (total > ctx->dp_bytes) {
        CU(ctx, stream_sync(ctx));
        cudaFree(ctx->d_dp);
        ctx->d_dp = nullptr;
        ctx->dp_bytes = 0;
        cudaError_t e = cudaMalloc(&ctx->d_dp, total);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SAILOR_E_NOMEM; }
        ctx->dp_bytes = total;
    }
    Bump bump{ctx->d_dp};
    double* d_tabs = bump.take<double>(tab_bytes / sizeof(double));
    uint32_t* d_vtabs = bump.take<uint32_t>(vtabs.size() + 1);
    DpResult* d_results = bump.take<DpResult>(n_problems);
    DpProblem* d_problems = bump.take<DpProblem>(n_problems);
    uint32_t* d_blk_problem = bump.take<uint32_t>(max_blocks + p_max + 16);
    uint32_t* d_blk_first = bump.take<uint32_t>(max_blocks + p_max + 16);
    DpVal* d_val0 = bump.take<DpVal>(max_entries);
    DpVal* d_val1 = bump.take<DpVal>(max_entries);
    uint8_t* d_choice = bump.take<uint8_t>(max_choice);
    sailor_dp_result* d_out = bump.take<sailor_dp_result>(SAILOR_K_MAX);
    unsigned long long* d_counters = bump.take<unsigned long long>(3);

    uint32_t launches = 0;
    {
        const int rc_up = upload_availability(ctx);
        if (rc_up) return rc_up;
    }
    CU(ctx, cudaEventRecord(ctx->ev0, ctx->stream));
    CU(ctx, cudaMemsetAsync(d_tabs, 0, tab_bytes, ctx->stream));
    CU(ctx, cudaMemsetAsync(d_counters, 0, 24, ctx->stream));
    if (!vtabs.empty())
        CU(ctx, cudaMemcpyAsync(d_vtabs, vtabs.data(), vtabs.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, ctx->stream));
    {
        const uint32_t grid = (uint32_t)(n_config < 4096 ? n_config : 4096);
        dp_tables_kernel<<<grid, DP_THREADS, 0, ctx->stream>>>(ctx->d_blob, d, (uint32_t)n_config, lay, d_tabs);
        CU(ctx, cudaGetLastError());
        ++launches;
    }
    // problems that have no entries still get their "no plan" result from the finish step
    std::vector<DpProblem> stage_buf;
    std::vector<uint32_t> blk_problem, blk_first;
    {
        stage_buf.clear();
        for (uint64_t j = 0; j < n_problems; ++j)
            if (!prob[j].n_lvl) stage_buf.push_back(prob[j]);
        if (!stage_buf.empty()) {
            CU(ctx, cudaMemcpyAsync(d_problems, stage_buf.data(), stage_buf.size() * sizeof(DpProblem), cudaMemcpyHostToDevice,
                                    ctx->stream));
            DpFinishParams fp;
            memset(&fp, 0, sizeof(fp));
            fp.blob = ctx->d_blob; fp.avail = ctx->d_avail; fp.sp = d; fp.problems = d_problems; fp.tabs = d_tabs; fp.vtabs = d_vtabs; fp.val[0] = d_val0; fp.val[1] = d_val1; fp.choice = d_choice;
            fp.results = d_results; fp.lay = lay; fp.n_problems = (uint32_t)stage_buf.size(); fp.T = T;
            dp_finish_kernel<<<(fp.n_problems + 127) / 128, 128, 0, ctx->stream>>>(fp);
            CU(ctx, cudaGetLastError());
            ++launches;
            CU(ctx, stream_sync(ctx));       // the staging vector is reused below
        }
    }
    for (const Batch& b : batches) {
        stage_buf.resize(b.count);
        blk_problem.clear();
        blk_first.clear();
        uint64_t val_off = 0, choice_off = 0;
        uint32_t max_p = 0;
        std::vector<uint64_t> blocks_upto(p_max + 2, 0);       // entries mode: blocks of problems deeper than a distance
        std::vector<uint64_t> dist_off(p_max + 2, 0);          // live mode: where the block list of a distance starts
        for (size_t j = 0; j < b.count; ++j) {
            DpProblem pb = prob[by_depth[b.first + j]];
            pb.val_off = val_off;
            pb.choice_off = choice_off;
            val_off += pb.n_lvl;
            choice_off += (uint64_t)pb.n_lvl * pb.P;
            stage_buf[j] = pb;
            max_p = pb.P > max_p ? pb.P : max_p;
            if (!all_live) {
                const uint32_t nb = (pb.n_lvl + DP_THREADS - 1) / DP_THREADS;
                for (uint32_t q = 0; q < nb; ++q) { blk_problem.push_back((uint32_t)j); blk_first.push_back(q * DP_THREADS); }
                for (uint32_t dist = 0; dist < pb.P; ++dist) blocks_upto[dist] += nb;
            }
        }
        std::vector<uint32_t> n_active(p_max + 1, 0), per_thread(p_max + 1, 1);
        // small problems only (no stage of any problem has more than a few blocks' worth of count vectors): a block
        // per problem runs all its stages in one launch
        bool block_per_problem = by_vector;
        for (size_t j = 0; block_per_problem && j < b.count; ++j) {
            const uint32_t pj = by_depth[b.first + j];
            for (uint32_t st = 0; st < prob[pj].P; ++st)
                if (live_cnt[live_off[pj] + st] > 8u * DP_THREADS) { block_per_problem = false; break; }
        }
        if (all_live && !block_per_problem) {                                        // per distance from the last stage: blocks before each problem
            for (uint32_t dist = 0; dist < max_p; ++dist) {
                dist_off[dist] = blk_problem.size();
                uint32_t blocks = 0;
                if (by_vector) {                               // small launches keep one vector per thread: more blocks
                    uint64_t vectors = 0;
                    for (size_t j = 0; j < b.count && prob[by_depth[b.first + j]].P > dist; ++j) {
                        const uint32_t pj = by_depth[b.first + j];
                        vectors += live_cnt[live_off[pj] + (prob[pj].P - 1 - dist)];
                    }
                    if (vectors >= 16ull * ctx->sm_count * DP_THREADS * DP_VEC_PER_THREAD) per_thread[dist] = DP_VEC_PER_THREAD;
                }
                const uint32_t per_block = DP_THREADS * per_thread[dist];
                for (size_t j = 0; j < b.count; ++j) {
                    const uint32_t pj = by_depth[b.first + j];
                    const DpProblem& pb = prob[pj];
                    if (pb.P <= dist) break;                   // sorted by depth
                    blk_problem.push_back(blocks);
                    blocks += (uint32_t)(((uint64_t)live_cnt[live_off[pj] + (pb.P - 1 - dist)] * live_mult + per_block - 1) / per_block);
                    ++n_active[dist];
                }
                blk_problem.push_back(blocks);
            }
            dist_off[max_p] = blk_problem.size();
            blk_first.assign(1, 0);                            // unused in this mode
        }
        CU(ctx, cudaMemcpyAsync(d_problems, stage_buf.data(), b.count * sizeof(DpProblem), cudaMemcpyHostToDevice, ctx->stream));
        if (!blk_problem.empty())
            CU(ctx, cudaMemcpyAsync(d_blk_problem, blk_problem.data(), blk_problem.size() * sizeof(uint32_t), cudaMemcpyHostToDevice,
                                    ctx->stream));
        if (!blk_first.empty())
            CU(ctx, cudaMemcpyAsync(d_blk_first, blk_first.data(), blk_first.size() * sizeof(uint32_t), cudaMemcpyHostToDevice,
                                    ctx->stream));
        DpLevelParams lp;
        memset(&lp, 0, sizeof(lp));
        lp.problems = d_problems; lp.blk_problem = d_blk_problem; lp.blk_first = d_blk_first; lp.tabs = d_tabs;
        lp.vtabs = d_vtabs;
        lp.val[0] = d_val0; lp.val[1] = d_val1; lp.choice = d_choice; lp.lay = lay; lp.T = T;
        if (block_per_problem) {
            if (T <= 4) dp_problem_kernel<4><<<(uint32_t)b.count, DP_THREADS, vt_len_max * 4, ctx->stream>>>(lp);
            else dp_problem_kernel<SAILOR_T_MAX><<<(uint32_t)b.count, DP_THREADS, vt_len_max * 4, ctx->stream>>>(lp);
            CU(ctx, cudaGetLastError());
            ++launches;
        }
        for (uint32_t dist = 0; dist < max_p && !block_per_problem; ++dist) {
            lp.dist = dist;
            if (all_live) {
                const uint32_t n_blk = blk_problem[dist_off[dist] + n_active[dist]];
                if (n_blk == 0) continue;
                lp.blk_prefix = d_blk_problem + dist_off[dist];
                lp.n_active = n_active[dist];
                lp.per_thread = per_thread[dist];
                if (by_vector && T <= 4) dp_level_vec_kernel<4><<<n_blk, DP_THREADS, vt_len_max * 4, ctx->stream>>>(lp);
                else if (by_vector) dp_level_vec_kernel<SAILOR_T_MAX><<<n_blk, DP_THREADS, vt_len_max * 4, ctx->stream>>>(lp);
                else dp_level_kernel<true><<<n_blk, DP_THREADS, 0, ctx->stream>>>(lp);
            } else {
                dp_level_kernel<false><<<(uint32_t)blocks_upto[dist], DP_THREADS, 0, ctx->stream>>>(lp);
            }
            CU(ctx, cudaGetLastError());
            ++launches;
        }
        DpFinishParams fp;
        memset(&fp, 0, sizeof(fp));
        fp.blob = ctx->d_blob; fp.avail = ctx->d_avail; fp.sp = d; fp.problems = d_problems; fp.tabs = d_tabs; fp.vtabs = d_vtabs; fp.val[0] = d_val0; fp.val[1] = d_val1; fp.choice = d_choice;
        fp.results = d_results; fp.lay = lay; fp.n_problems = (uint32_t)b.count; fp.T = T;
        dp_finish_kernel<<<(fp.n_problems + 127) / 128, 128, 0, ctx->stream>>>(fp);
        CU(ctx, cudaGetLastError());
        ++launches;
        CU(ctx, stream_sync(ctx));           // the host vectors are reused by the next batch
    }
    DpSelectParams sel;
    memset(&sel, 0, sizeof(sel));
    sel.results = d_results; sel.out = d_out; sel.counters = d_counters;
    sel.sp = d; sel.n_problems = (uint32_t)n_problems; sel.n_orders = n_orders; sel.k = k;
    sel.budget = o->budget_usd_per_iter; sel.min_rate = o->min_iters_per_s;
    dp_select_kernel<<<1, DP_SELECT_THREADS, 0, ctx->stream>>>(sel);
    CU(ctx, cudaGetLastError());
    ++launches;
    CU(ctx, cudaEventRecord(ctx->ev1, ctx->stream));
    unsigned long long counters[3] = {0, 0, 0};
    std::vector<sailor_dp_result> host_out(k);
    CU(ctx, cudaMemcpyAsync(counters, d_counters, sizeof(counters), cudaMemcpyDeviceToHost, ctx->stream));
    CU(ctx, cudaMemcpyAsync(host_out.data(), d_out, sizeof(sailor_dp_result) * k, cudaMemcpyDeviceToHost, ctx->stream));
    CU(ctx, stream_sync(ctx));
    if (counters[1] > k) return SAILOR_E_DEVICE;               // cannot happen; never copy past the caller's k records
    *n_found = (uint32_t)counters[1];
    memcpy(topk, host_out.data(), sizeof(sailor_dp_result) * counters[1]);
    if (stats) {
        stats->n_problems = n_problems;
        stats->n_solved = counters[0];
        stats->n_over_constraint = counters[2];
        stats->n_states = n_states;
        stats->workspace_used = largest;
        float ms = 0.f;
        CU(ctx, cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
        stats->kernel_ms = ms;
        stats->n_launches = launches;
        stats->n_batches = (uint32_t)batches.size();
        stats->n_unfinished = 0;
    }
    return SAILOR_OK;
}

// ---- search over plans with mixed replicas -------------------------------------------------------------

namespace {

// The combinations of `units` over T types with at most SAILOR_MIX_GROUPS_MAX non-empty types, in descending
// lexicographic order, one 64-bit word each (byte g = units on type g).
void list_combinations(uint32_t T, uint32_t units, std::vector<uint64_t>& out) {
    struct Rec {
        static void go(uint32_t T, uint32_t t, uint32_t left, uint32_t nonzero, uint64_t word, std::vector<uint64_t>& out) {
            if (t + 1 == T) {                                  // the last type takes what is left
                if (nonzero + (left ? 1u : 0u) <= SAILOR_MIX_GROUPS_MAX) out.push_back(word | ((uint64_t)left << (8 * t)));
                return;
            }
            for (uint32_t u = left + 1; u-- > 0;) {            // most units first
                const uint32_t nz = nonzero + (u ? 1u : 0u);
                if (nz > SAILOR_MIX_GROUPS_MAX) continue;
                go(T, t + 1, left - u, nz, word | ((uint64_t)u << (8 * t)), out);
            }
        }
    };
    Rec::go(T, 0, units, 0, 0, out);
}

struct MixedTables {
    MixedSpaceDesc desc;
    std::vector<uint64_t> combs;
    std::vector<uint64_t> flat_base;           // [n_config + 1]
    uint32_t n_config = 0;
};

int build_mixed_tables(const sailor_ctx* ctx, const sailor_mixed_space* s, MixedTables& mt) {
    if (!ctx || !s) return SAILOR_E_ARG;
    if (s->n_p == 0 || s->n_mbs == 0 || s->n_rc == 0 || s->n_d == 0 || s->granularity == 0) return SAILOR_E_ARG;
    if (s->n_p > SAILOR_NP_MAX || s->n_mbs > SAILOR_MBS_MAX || s->n_rc > 2 || s->n_d > SAILOR_ND_MAX || s->seg_max < 1 ||
        s->seg_max > SAILOR_SEG_MAX)
        return SAILOR_E_RANGE;
    const TabHdr& h = ctx->hdr;
    for (uint32_t i = 0; i < s->n_p; ++i)
        if (s->p_values[i] < 1 || s->p_values[i] > SAILOR_MIX_P_MAX) return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < s->n_mbs; ++i)
        if (s->mbs_idx[i] >= h.n_mbs) return SAILOR_E_RANGE;
    for (uint32_t i = 0; i < s->n_rc; ++i)
        if (s->rc_values[i] > 1) return SAILOR_E_RANGE;
    for (uint32_t g = 0; g < h.T; ++g)
        if (s->tp_idx_of_type[g] >= h.n_tp) return SAILOR_E_RANGE;
    MixedSpaceDesc& d = mt.desc;
    memset(&d, 0, sizeof(d));
    d.n_p = s->n_p; d.n_mbs = s->n_mbs; d.n_rc = s->n_rc; d.n_d = s->n_d; d.seg_max = s->seg_max; d.granularity = s->granularity;
    memcpy(d.p_values, s->p_values, sizeof(d.p_values));
    memcpy(d.mbs_idx, s->mbs_idx, sizeof(d.mbs_idx));
    memcpy(d.rc_values, s->rc_values, sizeof(d.rc_values));
    memcpy(d.tp_idx_of_type, s->tp_idx_of_type, sizeof(d.tp_idx_of_type));
    memcpy(d.d_values, s->d_values, sizeof(d.d_values));
    std::map<uint32_t, std::pair<uint32_t, uint32_t>> by_units;        // units -> (offset, count): degrees often share them
    for (uint32_t j = 0; j < s->n_d; ++j) {
        const uint32_t D = s->d_values[j];
        if (D < 1) return SAILOR_E_RANGE;
        const uint32_t units = mixed_units(s->granularity, D);
        if (units > SAILOR_MIX_UNITS_MAX) return SAILOR_E_RANGE;
        auto it = by_units.find(units);
        if (it == by_units.end()) {
            const uint32_t off = (uint32_t)mt.combs.size();
            list_combinations(h.T, units, mt.combs);
            it = by_units.emplace(units, std::make_pair(off, (uint32_t)mt.combs.size() - off)).first;
        }
        d.comb_off[j] = it->second.first;
        d.n_comb[j] = it->second.second;
    }
    const uint64_t n_config = (uint64_t)s->n_p * s->n_mbs * s->n_rc * s->n_d;
    if (n_config > (1u << 16)) return SAILOR_E_RANGE;
    mt.n_config = (uint32_t)n_config;
    mt.flat_base.assign(n_config + 1, 0);
    unsigned __int128 run = 0;
    for (uint32_t c = 0; c < n_config; ++c) {
        mt.flat_base[c] = (uint64_t)run;
        const MixedConfig k = mixed_config_of(d, c);
        const unsigned __int128 radix = (unsigned __int128)h.Z * d.n_comb[k.di];
        unsigned __int128 block = 1;
        for (uint32_t q = 0; q < k.nseg; ++q) {
            block *= radix;
            if (block >> 63) return SAILOR_E_RANGE;
        }
        run += block;
        if (run >> 63) return SAILOR_E_RANGE;
    }
    mt.flat_base[n_config] = (uint64_t)run;
    return SAILOR_OK;
}

}  // namespace

static int plan_mixed_impl(sailor_ctx* ctx, const sailor_mixed_space* s, const sailor_objective* o, uint32_t k,
                           sailor_mixed_result* topk, uint32_t* n_found, sailor_stats* stats) {
    if (!ctx || !s || !o || !topk || !n_found || k == 0) return SAILOR_E_ARG;
    if (k > SAILOR_K_MAX || o->kind > SAILOR_OBJ_MAX_THROUGHPUT_PER_USD) return SAILOR_E_RANGE;
    if (o->flags != 0 || o->budget_factor_over_cheapest > 0.0 || std::isnan(o->budget_usd_per_iter) ||
        std::isnan(o->min_iters_per_s) || std::isnan(o->budget_factor_over_cheapest))
        return SAILOR_E_ARG;
    MixedTables mt;
    int rc = build_mixed_tables(ctx, s, mt);
    if (rc) return rc;
    const uint64_t n_total = mt.flat_base[mt.n_config];
    DeviceGuard guard(ctx->device);
    const uint32_t R = ctx->hdr.R;
    const size_t smem = ctx->hdr.static_bytes + sizeof(unsigned long long) * MIXS_WARPS * R + sizeof(sailor_mixed_plan) * MIXS_WARPS;
    const uint64_t want_blocks = (n_total + MIXS_WARPS - 1) / MIXS_WARPS;
    const uint32_t grid = (uint32_t)std::min<uint64_t>(std::max<uint64_t>(want_blocks, 1), (uint64_t)ctx->sm_count * 4);
    const size_t total = padded(mt.combs.size() * 8) + padded(mt.flat_base.size() * 8) + padded(sizeof(Hit) * SAILOR_K_MAX * grid) +
                         padded(sizeof(sailor_mixed_result) * SAILOR_K_MAX) + padded(9 * 8) + 1024;
    if (total > ctx->mix_bytes) {
        CU(ctx, stream_sync(ctx));
        cudaFree(ctx->d_mix);
        ctx->d_mix = nullptr;
        ctx->mix_bytes = 0;
        cudaError_t e = cudaMalloc(&ctx->d_mix, total);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SAILOR_E_NOMEM; }
        ctx->mix_bytes = total;
    }
    Bump bump{ctx->d_mix};
    uint64_t* d_combs = bump.take<uint64_t>(mt.combs.size());
    uint64_t* d_base = bump.take<uint64_t>(mt.flat_base.size());
    Hit* d_partial = bump.take<Hit>((size_t)SAILOR_K_MAX * grid);
    sailor_mixed_result* d_results = bump.take<sailor_mixed_result>(SAILOR_K_MAX);
    unsigned long long* d_counters = bump.take<unsigned long long>(9);

    {
        const int rc_up = upload_availability(ctx);
        if (rc_up) return rc_up;
    }
    CU(ctx, cudaMemcpyAsync(d_combs, mt.combs.data(), mt.combs.size() * 8, cudaMemcpyHostToDevice, ctx->stream));
    CU(ctx, cudaMemcpyAsync(d_base, mt.flat_base.data(), mt.flat_base.size() * 8, cudaMemcpyHostToDevice, ctx->stream));
    CU(ctx, cudaMemsetAsync(d_counters, 0, 9 * 8, ctx->stream));
    CU(ctx, cudaMemsetAsync(d_counters + 6, 0x7f, 8, ctx->stream));           // the cheapest cost starts above every cost
    CU(ctx, cudaEventRecord(ctx->ev0, ctx->stream));
    MixedSearchParams mp;
    memset(&mp, 0, sizeof(mp));
    mp.blob = ctx->d_blob; mp.avail = ctx->d_avail; mp.cfg_flat_base = d_base; mp.combs = d_combs; mp.partial = d_partial;
    mp.counters = d_counters; mp.results = d_results; mp.sp = mt.desc; mp.n_config = mt.n_config; mp.k = k; mp.obj = o->kind;
    mp.n_partial = grid; mp.n_total = n_total; mp.budget = o->budget_usd_per_iter; mp.min_rate = o->min_iters_per_s;
    bool deep = false;                                           // pipelines of more than 32 stages in the space
    for (uint32_t i = 0; i < s->n_p; ++i) deep = deep || s->p_values[i] > 32;
    if (deep) plan_mixed_kernel<true><<<grid, MIXS_THREADS, smem, ctx->stream>>>(mp);
    else plan_mixed_kernel<false><<<grid, MIXS_THREADS, smem, ctx->stream>>>(mp);
    CU(ctx, cudaGetLastError());
    mixed_finish_kernel<<<1, MIXS_THREADS, smem, ctx->stream>>>(mp);
    CU(ctx, cudaGetLastError());
    CU(ctx, cudaEventRecord(ctx->ev1, ctx->stream));
    unsigned long long counters[9];
    std::vector<sailor_mixed_result> host_out(k);
    CU(ctx, cudaMemcpyAsync(counters, d_counters, sizeof(counters), cudaMemcpyDeviceToHost, ctx->stream));
    CU(ctx, cudaMemcpyAsync(host_out.data(), d_results, sizeof(sailor_mixed_result) * k, cudaMemcpyDeviceToHost, ctx->stream));
    CU(ctx, stream_sync(ctx));                                 // also: the host tables are pageable
    if (counters[7]) return SAILOR_E_DEVICE;
    if (counters[8] > k) return SAILOR_E_DEVICE;
    *n_found = (uint32_t)counters[8];
    memcpy(topk, host_out.data(), sizeof(sailor_mixed_result) * counters[8]);
    if (stats) {
        memset(stats, 0, sizeof(*stats));
        stats->n_total = counters[0];
        stats->n_invalid = counters[1];
        stats->n_oom = counters[2];
        stats->n_over_avail = counters[3];
        stats->n_over_constraint = counters[4];
        stats->n_feasible = counters[5];
        stats->budget_used = o->budget_usd_per_iter;
        double mc;
        memcpy(&mc, &counters[6], sizeof(mc));
        stats->min_feasible_cost = counters[5] ? mc : 0.0;
        CU(ctx, cudaEventElapsedTime(&stats->kernel_ms, ctx->ev0, ctx->ev1));
        stats->n_launches = 2;
        stats->n_configs = stats->n_configs_evaluated = mt.n_config;
    }
    return SAILOR_OK;
}

extern "C" int sailor_mixed_space_size(const sailor_ctx* ctx, const sailor_mixed_space* s, uint64_t* n_out) {
    if (!n_out) return SAILOR_E_ARG;
    try {
        MixedTables mt;
        const int rc = build_mixed_tables(ctx, s, mt);
        if (rc) return rc;
        *n_out = mt.flat_base[mt.n_config];
        return SAILOR_OK;
    } catch (const std::bad_alloc&) { return SAILOR_E_NOMEM; } catch (...) { return SAILOR_E_ARG; }
}

extern "C" int sailor_mixed_decode(const sailor_ctx* ctx, const sailor_mixed_space* s, uint64_t flat, sailor_mixed_plan* out) {
    if (!out) return SAILOR_E_ARG;
    try {
        MixedTables mt;
        const int rc = build_mixed_tables(ctx, s, mt);
        if (rc) return rc;
        if (flat >= mt.flat_base[mt.n_config]) return SAILOR_E_RANGE;
        const uint32_t c = (uint32_t)(std::upper_bound(mt.flat_base.begin(), mt.flat_base.end(), flat) - mt.flat_base.begin()) - 1;
        const MixedConfig k = mixed_config_of(mt.desc, c);
        const uint64_t radix = (uint64_t)ctx->hdr.Z * mt.desc.n_comb[k.di];
        uint64_t rem = flat - mt.flat_base[c];
        uint32_t digit[SAILOR_SEG_MAX] = {0, 0, 0, 0};
        for (uint32_t q = k.nseg; q-- > 0;) { digit[q] = (uint32_t)(rem % radix); rem /= radix; }
        memset(out, 0, sizeof(*out));
        out->P = (uint8_t)k.P; out->mbs_idx = (uint8_t)k.mi; out->rc = (uint8_t)k.rc; out->D = (uint16_t)k.D;
        for (uint32_t i = 0; i < k.P; ++i) mixed_build_stage(mt.desc, k, ctx->hdr.T, mt.combs.data(), digit, i, &out->stage[i]);
        return SAILOR_OK;
    } catch (const std::bad_alloc&) { return SAILOR_E_NOMEM; } catch (...) { return SAILOR_E_ARG; }
}

extern "C" int sailor_plan_mixed(sailor_ctx* ctx, const sailor_mixed_space* s, const sailor_objective* o, uint32_t k,
                                 sailor_mixed_result* topk, uint32_t* n_found, sailor_stats* stats) {
    try {
        return plan_mixed_impl(ctx, s, o, k, topk, n_found, stats);
    } catch (const std::bad_alloc&) { return SAILOR_E_NOMEM; } catch (...) { return SAILOR_E_ARG; }
}

// ---- sustained issue rates (measurement) ---------------------------------------------------------------

extern "C" int sailor_measure_issue_rates(int cuda_device, void* cuda_stream, uint32_t repeats, sailor_issue_rates* out) {
    if (!out || repeats == 0) return SAILOR_E_ARG;
    memset(out, 0, sizeof(*out));
    DeviceGuard guard(cuda_device);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cuda_device) != cudaSuccess) return SAILOR_E_CUDA;
    double* sink = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaMalloc(&sink, sizeof(double)) != cudaSuccess) return SAILOR_E_CUDA;
    int rc = SAILOR_OK;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) rc = SAILOR_E_CUDA;
    const uint32_t grid = (uint32_t)prop.multiProcessorCount * 4, iters = 2048;
    const uint64_t per_run = (uint64_t)grid * (PEAK_THREADS / 32) * iters * PEAK_CHAINS * PEAK_ROUNDS;
    float best[3] = {0.f, 0.f, 0.f};
    for (int kind = 0; kind < 3 && rc == SAILOR_OK; ++kind) {
        for (uint32_t r = 0; r <= repeats && rc == SAILOR_OK; ++r) {        // run 0 warms up
            cudaEventRecord(e0, stream);
            // multipliers just below one and small addends keep every chain finite for any run length
            if (kind == PEAK_FFMA) issue_stream_kernel<PEAK_FFMA><<<grid, PEAK_THREADS, 0, stream>>>(iters, 0.999f, 0.5f, 0, 0, 0.0, sink);
            else if (kind == PEAK_IMAD) issue_stream_kernel<PEAK_IMAD><<<grid, PEAK_THREADS, 0, stream>>>(iters, 0.f, 0.f, 2654435761u, 12345u, 0.0, sink);
            else issue_stream_kernel<PEAK_DADD><<<grid, PEAK_THREADS, 0, stream>>>(iters, 0.f, 0.f, 0, 0, 0.25, sink);
            cudaEventRecord(e1, stream);
            float ms = 0.f;
            if (cudaGetLastError() != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
                cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess)
                rc = SAILOR_E_CUDA;
            else if (r > 0 && ms > 0.f && (best[kind] == 0.f || ms < best[kind])) best[kind] = ms;
        }
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(sink);
    if (rc) return rc;
    out->ffma_ms = best[0]; out->imad_ms = best[1]; out->dadd_ms = best[2];
    out->ffma_warp_inst_per_s = best[0] > 0.f ? (double)per_run / (best[0] * 1e-3) : 0.0;
    out->imad_warp_inst_per_s = best[1] > 0.f ? (double)per_run / (best[1] * 1e-3) : 0.0;
    out->dadd_warp_inst_per_s = best[2] > 0.f ? (double)per_run / (best[2] * 1e-3) : 0.0;
    out->sm_count = (uint32_t)prop.multiProcessorCount;
    out->warp_inst_per_run = per_run;
    return SAILOR_OK;
}

// ---- entry points that build host-side tables: no exception may cross the C boundary -------------------

#define SAILOR_NO_THROW(call)                              \
    try {                                                  \
        return call;                                       \
    } catch (const std::bad_alloc&) {                      \
        return SAILOR_E_NOMEM;                             \
    } catch (...) {                                        \
        return SAILOR_E_ARG;                               \
    }

extern "C" {

int sailor_create(const sailor_model* m, const sailor_profile* p, const sailor_cluster* c, int cuda_device,
                  void* cuda_stream, sailor_ctx** out) {
    SAILOR_NO_THROW(create_impl(m, p, c, cuda_device, cuda_stream, out))
}

int sailor_plan_range(sailor_ctx* ctx, const sailor_space* s, const sailor_objective* o, uint64_t flat_lo,
                      uint64_t flat_hi, uint32_t k, sailor_result* topk, uint32_t* n_found, sailor_stats* stats) {
    SAILOR_NO_THROW(plan_range_impl(ctx, s, o, flat_lo, flat_hi, k, topk, n_found, stats))
}

int sailor_plan_dp(sailor_ctx* ctx, const sailor_space* s, const sailor_zone_order* orders, uint32_t n_orders,
                   const sailor_objective* o, uint64_t workspace_bytes, uint32_t k, sailor_dp_result* topk,
                   uint32_t* n_found, sailor_dp_stats* stats) {
    SAILOR_NO_THROW(plan_dp_impl(ctx, s, orders, n_orders, o, workspace_bytes, k, topk, n_found, stats))
}

}  // extern "C"
