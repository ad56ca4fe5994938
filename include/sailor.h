/*
 * sailor.h — C ABI of the batched plan simulator and plan search (CUDA, sm_100a).
 *
 * The library evaluates candidate training-job configurations with the Sailor
 * simulator (Sailor, SOSP'25, Sec. 4.3: memory footprint, 1F1B iteration time,
 * cost per iteration) and reduces a whole search space to the best plan and the
 * top-k under an objective and a constraint (Sec. 4.2, last two paragraphs of the
 * planner overview).  Every candidate is simulated on the GPU; there is no CPU
 * fallback.  All functions return 0 on success and a negative SAILOR_E_* code on
 * failure; none throws, aborts or prints.
 *
 * Conventions
 *   P      pipeline stages          D    data-parallel degree (same for all stages, H3)
 *   tp     tensor-parallel degree   mbs  microbatch size
 *   gbs    global batch size        N_b  = gbs / (D * mbs), microbatches per pipeline
 *   T      GPU types                Z    zones; a "digit" d = zone * T + type
 *   kinds  layer kinds: 0 = EMBED, 1 = BLOCK, 2 = HEAD
 *
 * Arithmetic.  Bytes and counts are unsigned integers (exact).  Times and costs
 * are IEEE binary64 evaluated in one fixed order without fused multiply-add:
 *   f_i   = sum over the layers of stage i (stage order) of fwd[kind][g_i][tp_i][mbs]
 *   b_i   = same over bwd, then + f_i when recomputation is on
 *   u_i   = same over upd[kind][g_i][tp_i]
 *   c_i   = alpha(link_i) + (double)p2p_bytes[mbs] * inv_bw(link_i), 0 for the last stage
 *           (with a bandwidth polynomial: alpha + m / (((p3*m + p2)*m + p1)*m + p0))
 *   t_i   = (f_i + b_i) + 2 * c_i
 *   T_pp  = (t_0 + t_1 + ... left to right) + (double)N_b * max_i t_i
 *   sync_i= D == 1 ? 0 : ((2(D-1))/D * (double)gradbytes_i) * inv_bw_dp(i) + (2(D-1)) * alpha_dp(i)
 *           (with a polynomial: "* inv_bw" becomes "/ bandwidth((double)gradbytes_i / D)")
 *   T_iter= (T_pp + max_i sync_i) + max_i u_i                          (Sec. 4.3, Sec. 4.2.2)
 *   rate  = sum_i (double)(D * tp_i) * (price_per_hour[z_i][g_i] / 3600)   left to right
 *   C_comm= sum over stage boundaries that cross zones of
 *           (double)(2 * N_b * D * p2p_bytes[mbs]) * egress[z_i][z_{i+1}]  left to right
 *   C_iter= rate * T_iter + C_comm                                      (Sec. 4.3, Sec. 4.2.3)
 *
 * Threading.  A context is not thread-safe; use one context per host thread.  Different
 * contexts may be used from different threads at the same time (the library's few process-wide
 * flags are atomic).  The library reads no environment variable and keeps no other global state.
 */
#ifndef SAILOR_H
#define SAILOR_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- limits --------------------------------------------------------------------------- */
#define SAILOR_KINDS      3     /* EMBED, BLOCK, HEAD                                       */
#define SAILOR_T_MAX      8     /* GPU types                                                */
#define SAILOR_Z_MAX      8     /* zones                                                    */
#define SAILOR_TP_MAX     8     /* entries of tp_values                                     */
#define SAILOR_MBS_MAX    16    /* entries of mbs_values                                    */
#define SAILOR_P_MAX      96    /* pipeline stages in one plan                              */
#define SAILOR_RUN_MAX    16    /* runs in a plan record                                    */
#define SAILOR_SEG_MAX    4     /* segments the enumerator varies per plan                  */
#define SAILOR_K_MAX      32    /* top-k                                                    */
#define SAILOR_NP_MAX     32    /* entries of sailor_space.p_values                         */
#define SAILOR_ND_MAX     32    /* entries of sailor_space.d_values                         */

/* ---- error codes ---------------------------------------------------------------------- */
#define SAILOR_OK          0
#define SAILOR_E_ARG      (-1)  /* null pointer, zero k, inconsistent sizes, bad record      */
#define SAILOR_E_RANGE    (-2)  /* an index or a size is outside a table or a limit above    */
#define SAILOR_E_CUDA     (-3)  /* a CUDA call failed; see sailor_last_cuda_error            */
#define SAILOR_E_NOMEM    (-4)  /* host or device allocation failed                          */
#define SAILOR_E_DEVICE   (-5)  /* a kernel reported an internal fault (bounded wait ran out)
                                   during THIS call; the flag is cleared with the call, the
                                   context stays usable and the next call starts clean        */

/* ---- status bits of one simulated plan ------------------------------------------------- */
#define SAILOR_ST_INVALID          1u   /* gbs % (D*mbs) != 0, tp > gpus_per_node, heads % tp != 0 (H1) */
#define SAILOR_ST_OVER_AVAIL       2u   /* needs more GPUs of some (zone, type) than available           */
#define SAILOR_ST_OOM              4u   /* some stage's peak memory exceeds its GPU's capacity (H2)     */
#define SAILOR_ST_BAD_RECORD       32u  /* device-side record failed its bounds checks; nothing read    */
/* A budget or a throughput floor belongs to a search, not to a plan: sailor_simulate knows neither, so
 * no status bit exists for them; a search counts such candidates in sailor_stats.n_over_constraint. */

/* ---- inputs --------------------------------------------------------------------------- */

/* Training job (Sec. 4: "model training specifications").  Layers are n_blocks identical
 * BLOCK layers, preceded by one EMBED layer when has_embed and followed by one HEAD layer
 * when has_head.  A plan with P stages gives stage i  n_blocks / P  blocks, plus one more
 * for the first n_blocks % P stages; EMBED goes to stage 0, HEAD to stage P-1. */
typedef struct sailor_model {
    uint32_t n_blocks;          /* >= 1                                                     */
    uint32_t has_embed;         /* 0 / 1                                                    */
    uint32_t has_head;          /* 0 / 1                                                    */
    uint32_t heads;             /* attention heads; tp must divide it                       */
    uint64_t gbs;               /* global batch size, never changed by the planner          */
    uint32_t mul_factor;        /* copies of each parameter (weights, grads, optimizer), Sec. 4.3 */
    uint32_t dtype_size;        /* bytes per parameter copy                                 */
    uint32_t grad_dtype_size;   /* bytes per gradient element sent in the all-reduce        */
    uint32_t _pad;
} sailor_model;

/* Per-layer profile (Sec. 4.1, training job profiling).  All pointers are HOST arrays,
 * row-major in the index order shown, copied by sailor_create. */
typedef struct sailor_profile {
    uint32_t n_types, n_tp, n_mbs, _pad;
    uint32_t tp_values[SAILOR_TP_MAX];    /* tensor-parallel degree of each tp index        */
    uint32_t mbs_values[SAILOR_MBS_MAX];  /* microbatch size of each mbs index              */
    const double*   fwd;        /* [kind][type][tp][mbs] seconds, finite, >= 0              */
    const double*   bwd;        /* [kind][type][tp][mbs] seconds                            */
    const double*   upd;        /* [kind][type][tp]      seconds                            */
    const uint64_t* params;     /* [kind] parameters of one layer                           */
    const uint64_t* act_saved;  /* [kind][tp][mbs] bytes kept per in-flight microbatch      */
    const uint64_t* act_ckpt;   /* [kind][tp][mbs] bytes kept when recomputation is on      */
    const uint64_t* act_work;   /* [kind][tp][mbs] transient working bytes                  */
    const uint64_t* p2p_bytes;  /* [mbs] bytes one microbatch sends to the next stage       */
} sailor_profile;

/* Cluster (Sec. 4: quotas, prices; Sec. 4.1, cluster profiling).  A link is a degree-1
 * time model  time(m) = alpha + m * inv_bw  (seconds, seconds per byte).  HOST arrays. */
typedef struct sailor_cluster {
    uint32_t n_types, n_zones;
    const uint64_t* capacity;        /* [type] bytes of GPU memory                           */
    const uint64_t* reserved;        /* [type] bytes unavailable to the job                  */
    const uint32_t* gpus_per_node;   /* [type]                                               */
    const double*   price_per_hour;  /* [zone][type] USD per GPU-hour                        */
    const double*   intra_alpha;     /* [zone][type] link inside one node                    */
    const double*   intra_inv_bw;    /* [zone][type]                                         */
    const double*   inter_alpha;     /* [zone][type] link between nodes of one zone          */
    const double*   inter_inv_bw;    /* [zone][type]                                         */
    const double*   zone_alpha;      /* [zone][zone] link between zones (diagonal unused)    */
    const double*   zone_inv_bw;     /* [zone][zone]                                         */
    const double*   egress;          /* [zone][zone] USD per byte sent from row to column    */
    /* Optional message-size-dependent bandwidth (Sec. 4.1: a polynomial fitted to measured
     * bandwidth per link).  Four coefficients per link: bandwidth(m) = p0 + p1 m + p2 m^2 + p3 m^3
     * bytes/s for a message of m bytes (Horner, binary64), all >= 0 and p0 > 0.  A link with a
     * polynomial takes  alpha + m / bandwidth(m)  and ignores its inv_bw; the ring all-reduce
     * evaluates the bandwidth at its chunk size gradbytes / D.  NULL = constant bandwidth. */
    const double*   intra_bw_poly;   /* [zone][type][4] or NULL                               */
    const double*   inter_bw_poly;   /* [zone][type][4] or NULL                               */
    const double*   zone_bw_poly;    /* [zone][zone][4] or NULL                               */
} sailor_cluster;

/* One plan, stages run-length encoded: run r covers n_stages consecutive stages that share
 * (type, zone, tp).  sum of n_stages == P.  72 bytes; arrays of records must be 8-byte aligned. */
typedef struct sailor_run {
    uint8_t type, zone, tp_idx, n_stages;
} sailor_run;

typedef struct sailor_plan_rec {
    uint8_t  P;                 /* 1 .. SAILOR_P_MAX                                        */
    uint8_t  mbs_idx;
    uint8_t  rc;                /* 1 = activation recomputation                             */
    uint8_t  n_runs;            /* 1 .. SAILOR_RUN_MAX                                      */
    uint16_t D;                 /* >= 1                                                     */
    uint16_t _pad;
    sailor_run run[SAILOR_RUN_MAX];
} sailor_plan_rec;

/* Search space of sailor_plan.  Flat index, digits from low to high:
 *   seg[nseg-1], ..., seg[0]   radix T*Z each, digit = zone*T + type
 *   d_values index, rc_values index, tp_idx index, mbs_idx index
 * and the sub-spaces of the entries of p_values are concatenated in that order.
 * nseg = min(P, seg_max); stage i belongs to segment floor(i * nseg / P). */
typedef struct sailor_space {
    uint32_t n_p, n_mbs, n_tp, n_rc, n_d, seg_max;
    uint8_t  p_values[SAILOR_NP_MAX];
    uint8_t  mbs_idx[SAILOR_MBS_MAX];
    uint8_t  tp_idx[SAILOR_TP_MAX];
    uint8_t  rc_values[2];
    uint8_t  _pad[6];
    uint16_t d_values[SAILOR_ND_MAX];
} sailor_space;

#define SAILOR_OBJ_MAX_THROUGHPUT         0   /* minimise T_iter          */
#define SAILOR_OBJ_MIN_COST               1   /* minimise C_iter          */
#define SAILOR_OBJ_MAX_THROUGHPUT_PER_USD 2   /* minimise T_iter * C_iter */

#define SAILOR_FLAG_EVAL_ALL 1u  /* compute time and cost of every candidate, skipping nothing;
                                    results are identical with or without it                */

/* The planner's pruning heuristics as search modes (Sec. 4.2.1).  They change what is searched, so
 * the result may differ from the exhaustive search; sailor_stats says how much was left out.
 *
 * SAILOR_FLAG_DEGREE_ORDER (H3, H4).  A group is a configuration without its data-parallel degree:
 * (P, mbs, tp, rc).  Inside every group the degrees of d_values are tried from the largest down
 * when kind is MAX_THROUGHPUT (H3) and from the smallest up when it is MIN_COST (H4).  Degrees
 * with no feasible plan are passed over until the first feasible one; from then on the next degree
 * is tried only while the group's best score at the last degree was strictly better than at the
 * degree before.  The degree at which improvement stops has been evaluated and its plans compete
 * for the top-k; the group's remaining degrees are never looked at (n_skipped).  Whole-space
 * searches only; E_ARG with MAX_THROUGHPUT_PER_USD, with SAILOR_FLAG_EVAL_ALL, with a sub-range,
 * and in sailor_plan_noalloc.  With budget_factor_over_cheapest each of the two passes applies the
 * order of its own objective.  On the device the groups advance together: one launch per
 * position in the degree order evaluates that degree of every group still going.
 *
 * SAILOR_FLAG_MIN_TP_ONLY (H2, taken one step further).  The memory check already drops
 * tensor-parallel degrees that do not fit, which is H2 as printed.  This mode also drops a plan
 * when some smaller degree of tp_idx gives a valid plan in which every stage fits, so that of the
 * plans that differ only in tp the one with the smallest fitting degree remains.  Dropped plans
 * are counted in n_pruned_tp: after invalid and out of memory, before availability. */
#define SAILOR_FLAG_DEGREE_ORDER 2u
#define SAILOR_FLAG_MIN_TP_ONLY  4u

/* SAILOR_FLAG_F32_SCREEN.  Every candidate is first evaluated in binary32 (from tables rounded once per
 * configuration); a prefix with all its last digits is evaluated again in binary64, exactly as without the flag,
 * only when its best binary32 score comes within 1e-4 (relative) of the score a candidate must beat to enter the
 * top-k, or its cheapest binary32 cost within 1e-4 of the cheapest cost known.  The binary32 evaluation is off by
 * less than 1.4e-5 (relative; at most 96 stages), so the returned plans, scores, counts and min_feasible_cost are
 * the ones the search returns without the flag, bit for bit; only the time differs.  Searches without a budget, a
 * throughput floor or a budget factor only, and not with SAILOR_FLAG_DEGREE_ORDER (E_ARG); not in
 * sailor_plan_noalloc. */
#define SAILOR_FLAG_F32_SCREEN   8u

typedef struct sailor_objective {
    uint32_t kind;
    uint32_t flags;
    double   budget_usd_per_iter;          /* <= 0: none                                    */
    double   min_iters_per_s;              /* <= 0: none                                    */
    double   budget_factor_over_cheapest;  /* > 0: first find the cheapest feasible plan
                                              (MIN_COST, no budget), then search with budget
                                              = factor * that cost (two passes)             */
} sailor_objective;

typedef struct sailor_result {
    uint64_t flat;
    double   t_iter;
    double   cost;
    uint64_t peak_mem;
    double   score;
    uint32_t status;
    uint32_t _pad;
    sailor_plan_rec plan;
} sailor_result;

/* Every candidate that was looked at falls in exactly one class: the first of invalid, oom,
 * pruned_tp (SAILOR_FLAG_MIN_TP_ONLY), over_avail, over_constraint (budget or throughput) that
 * applies, else feasible.  n_total is their sum; n_total + n_skipped is the size of the space. */
typedef struct sailor_stats {
    uint64_t n_total, n_invalid, n_oom, n_over_avail, n_over_constraint, n_feasible;
    double   budget_used;       /* the budget the (last) pass ran with; <= 0 if none         */
    double   min_feasible_cost; /* smallest C_iter among the feasible candidates; 0 if none */
    float    kernel_ms;         /* device time of the search kernels (CUDA events)          */
    uint32_t n_launches;        /* kernels launched by this call                            */
    uint64_t n_pruned_tp;       /* dropped because a smaller tensor-parallel degree fits     */
    uint64_t n_skipped;         /* candidates of configurations early termination never reached */
    uint32_t n_configs;         /* configurations (P, mbs, tp, rc, D) of the space           */
    uint32_t n_configs_evaluated;   /* of which looked at (all of them without DEGREE_ORDER) */
    float    h2d_ms;            /* device time of the last availability upload to device memory
                                   (CUDA events around the copy; sailor_plan itself carries the
                                   snapshot in its launch parameters and needs no such copy: the
                                   entry points that read it through a pointer trigger one)     */
    float    d2h_ms;            /* device time of this call's result read-back; 0 where the
                                   kernel writes the results straight into pinned host memory
                                   (sailor_plan, sailor_plan_range)                             */
} sailor_stats;

typedef struct sailor_ctx sailor_ctx;     /* opaque; owns device copies of the tables       */

/* ---- entry points --------------------------------------------------------------------- */

/* Build a context on `cuda_device`.  Copies and validates the tables (HOST pointers),
 * uploads them, and precomputes on the device the left-to-right layer sums every stage
 * composition needs.  `cuda_stream` is a cudaStream_t (NULL = default stream) on which all
 * later work of this context is enqueued.  Availability starts at zero everywhere.
 * Errors: E_ARG (null, n_types mismatch, zero sizes, non-finite or negative table entry),
 * E_RANGE (a size beyond a limit), E_CUDA, E_NOMEM. */
int sailor_create(const sailor_model* m, const sailor_profile* p, const sailor_cluster* c,
                  int cuda_device, void* cuda_stream, sailor_ctx** out);

int sailor_destroy(sailor_ctx* ctx);      /* NULL is accepted                               */

/* Replace the availability snapshot (Sec. 4: "current availability of hardware resources").
 * `avail` is a HOST array [zone][type] of GPU counts, copied before the call returns.  It is the only
 * per-snapshot input: a search carries it to the device in its launch parameters; the device copy read by
 * sailor_simulate*, sailor_plan_dp and sailor_plan_mixed is refreshed when one of them is next called. */
int sailor_set_availability(sailor_ctx* ctx, const uint16_t* avail);

/* Simulate n explicit plans (Sec. 4.3).  Inputs and outputs are all HOST pointers when
 * on_device == 0 (copied both ways, stream synchronised before return) or all DEVICE
 * pointers when on_device == 1 (work is only enqueued on the context's stream).  Outputs are
 * arrays of n; any of them may be NULL.  t_iter and cost are NaN when SAILOR_ST_INVALID
 * or SAILOR_ST_BAD_RECORD is set; peak_mem is the maximum over stages of the per-GPU peak
 * (with N_b taken as floor(gbs / (D*mbs))).  A different tp per run is accepted (Sec. 4.4).
 * Host batches go through the device in chunks (2^19 records or 64 MB of records, whichever is less), results
 * coming back while the next chunk goes in; the library stages at most three chunks at a time, whatever n is.
 * Records are checked on the device, by the kernel that reads them.
 * Errors: E_ARG (null ctx/plans, unaligned plans), E_RANGE (host records only: an index
 * outside its table, n_runs or P outside limits, run lengths not summing to P; the outputs are
 * written all the same, the refused records with SAILOR_ST_BAD_RECORD and NaN), E_CUDA. */
int sailor_simulate(sailor_ctx* ctx, const sailor_plan_rec* plans, uint64_t n, int on_device,
                    double* t_iter, uint64_t* peak_mem, double* cost, uint32_t* status);

/* Number of candidates in a space (host arithmetic).  E_RANGE if it overflows 2^63. */
int sailor_space_size(const sailor_ctx* ctx, const sailor_space* s, uint64_t* n_out);

/* Flat index -> plan record (host arithmetic), the inverse of the enumeration order. */
int sailor_decode(const sailor_ctx* ctx, const sailor_space* s, uint64_t flat,
                  sailor_plan_rec* out);

/* Search the whole space (Sec. 4.2: evaluate candidates, keep those within the constraint,
 * order by the objective, return the best).  Candidates are generated on the device from
 * their flat index.  `topk` is a HOST array of k records, filled best first in
 * (score, flat) ascending order; *n_found <= k is how many are feasible.  An empty
 * feasible set is not an error.  `stats` may be NULL.  Synchronises the stream.
 * Errors: E_ARG (null, k == 0, empty radix list), E_RANGE (k > SAILOR_K_MAX, an index
 * outside its table, P > SAILOR_P_MAX, seg_max outside 1..SAILOR_SEG_MAX), E_CUDA, E_DEVICE. */
int sailor_plan(sailor_ctx* ctx, const sailor_space* s, const sailor_objective* o,
                uint32_t k, sailor_result* topk, uint32_t* n_found, sailor_stats* stats);

/* Same over the candidates with flat index in [flat_lo, flat_hi) only, so that a space can
 * be split over several GPUs and the per-range top-k lists merged by (score, flat).
 * With budget_factor_over_cheapest > 0 the cheapest plan is searched in this range only;
 * a sharded caller runs the MIN_COST pass itself and passes an explicit budget. */
int sailor_plan_range(sailor_ctx* ctx, const sailor_space* s, const sailor_objective* o,
                      uint64_t flat_lo, uint64_t flat_hi,
                      uint32_t k, sailor_result* topk, uint32_t* n_found, sailor_stats* stats);

/* Search without allocating.  (The paper has no counterpart: this entry point exists for the
 * sake of callers, not of the method.)
 *
 * sailor_plan allocates device memory whenever it meets a space it has not cached (two
 * cudaMalloc / cudaFree pairs for the per-configuration index arrays).  Some callers cannot
 * afford or are not allowed that: a re-planning loop inside a training process whose memory
 * pool already owns the whole GPU, where a further cudaMalloc fails; a latency-critical
 * controller for which cudaMalloc's device-wide synchronisation stalls every other stream;
 * a thread that runs while another thread of the process captures a stream in the global
 * capture mode, during which cudaMalloc is an error.  This variant computes exactly what
 * sailor_plan computes (whole space, same results, same statistics) but calls no cudaMalloc,
 * cudaFree or any other allocating routine: all of its working memory (work counter,
 * statistics, per-block top-k lists, result records, per-configuration index arrays) lies in
 * one array of about 0.6 MB that is part of the library image, so every GPU that loads the
 * library holds it until the process exits.  The context must already exist (sailor_create
 * allocates; call it at set-up).
 *
 * Limit: at most SAILOR_NOALLOC_CONFIG_MAX configurations, i.e.
 * n_p * n_mbs * n_tp * n_rc * n_d <= 4096; a larger space returns SAILOR_E_RANGE and nothing
 * is launched.  Other errors as sailor_plan.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call before any stream capture begins.
 * All calls, from every context on a device, share the one array: it keeps the previous
 * call's contents (the counters are cleared at the start of each call), and two calls that
 * overlap on the GPU (different streams or threads) race on it and return garbage.  Issue
 * them one after the other. */
#define SAILOR_NOALLOC_CONFIG_MAX 4096
int sailor_plan_noalloc(sailor_ctx* ctx, const sailor_space* s, const sailor_objective* o, uint32_t k,
                        sailor_result* topk, uint32_t* n_found, sailor_stats* stats);

/* ---- plans whose stages mix GPU types among their replicas (Sec. 4.2 problem statement, Sec. 4.3) ----
 *
 * In the paper a stage has D replicas, each with its own (GPU type, tp), all in one zone (H1, H5).
 * A stage lists its replicas as up to SAILOR_MIX_GROUPS_MAX groups of `count` equal replicas; the
 * counts of a stage add up to D.  Readings where the paper is silent:
 *   - replicas are numbered group after group and pipeline k is replica k of every stage; every
 *     pipeline processes N_b = gbs / (D * mbs) microbatches; T_pp(k) = sum_i t_i + N_b * max_i t_i over
 *     pipeline k's own stages; T_iter = (max_k T_pp(k) + max_i sync_i) + max update;
 *   - a message between neighbouring replicas stays inside a node only when both have the same GPU
 *     type and their two groups fit one node together (count*tp + count'*tp' <= gpus_per_node);
 *     across zones it takes the zone link, otherwise the slower of the two types' inter-node times;
 *   - a stage's all-reduce moves the largest gradient shard among its groups (the smallest tp); one
 *     group that fits a node (D*tp <= gpus_per_node) uses the intra-node link, otherwise every
 *     group's inter-node link carries the ring and the slowest sets the time;
 *   - memory is checked per group; the update time is the largest over stages and groups; the price
 *     rate adds (double)(count*tp) * price per second group after group, stage after stage.
 * A plan with one group in every stage gives bit-identical results to sailor_simulate. */
#define SAILOR_MIX_P_MAX       96    /* the deepest pipeline of the plain simulator's workloads */
#define SAILOR_MIX_GROUPS_MAX  4

typedef struct sailor_replica_group {
    uint8_t  type, tp_idx;
    uint16_t count;                     /* replicas in the group, >= 1                               */
} sailor_replica_group;

typedef struct sailor_mixed_stage {
    uint8_t  zone, n_groups;            /* 1 .. SAILOR_MIX_GROUPS_MAX                                 */
    uint16_t _pad;
    sailor_replica_group group[SAILOR_MIX_GROUPS_MAX];
} sailor_mixed_stage;

typedef struct sailor_mixed_plan {      /* 1928 bytes (only the first P stages are read); 8-byte aligned */
    uint8_t  P;                         /* 1 .. SAILOR_MIX_P_MAX                                      */
    uint8_t  mbs_idx, rc, _pad;
    uint16_t D;                         /* >= 1                                                       */
    uint16_t _pad2;
    sailor_mixed_stage stage[SAILOR_MIX_P_MAX];
} sailor_mixed_plan;

/* Simulate n such plans.  Pointers, outputs, NULLs, on_device and errors as sailor_simulate.
 * SAILOR_ST_INVALID also covers a stage whose counts do not add up to D or a group with count 0;
 * SAILOR_ST_BAD_RECORD an index outside its table or n_groups / P outside their limits. */
int sailor_simulate_mixed(sailor_ctx* ctx, const sailor_mixed_plan* plans, uint64_t n, int on_device,
                          double* t_iter, uint64_t* peak_mem, double* cost, uint32_t* status);

/* The same for records cut short, so that a batch of shallow plans need not carry SAILOR_MIX_P_MAX stages each:
 * record j starts at (const char*)plans + j * record_bytes and holds the 8-byte head of a sailor_mixed_plan and its
 * first (record_bytes - 8) / sizeof(sailor_mixed_stage) stages.  record_bytes is a multiple of 8 from 32 to
 * sizeof(sailor_mixed_plan), else SAILOR_E_ARG.  A plan with more stages than its record holds is refused
 * (host records: SAILOR_E_RANGE; device records: SAILOR_ST_BAD_RECORD and NaN for that plan). */
int sailor_simulate_mixed_strided(sailor_ctx* ctx, const void* plans, uint64_t n, uint32_t record_bytes, int on_device,
                                  double* t_iter, uint64_t* peak_mem, double* cost, uint32_t* status);

/* ---- searching over such plans (Sec. 4.2.2 "Implementation": per stage, the planner generates the resource
 * combinations of different GPU types that give the stage its D replicas) ---------------------------------
 *
 * A combination splits the D replicas of a stage over the GPU types.  To keep their number bounded the split is made
 * in `granularity` equal parts when granularity divides D (a part = D / granularity replicas), else replica by
 * replica: units(D) = granularity or D (at most SAILOR_MIX_UNITS_MAX), and a combination is a tuple (u_0 .. u_{T-1})
 * of units per type that add up to units(D), at most SAILOR_MIX_GROUPS_MAX of them non-zero.  Combinations are
 * numbered in descending lexicographic order of the tuple (everything on type 0 first; with one unit, combination c
 * is "everything on type c").  A stage built from a combination lists its non-empty types in ascending order: group
 * q = the q-th such type, count = units * D / units(D), tensor-parallel degree tp_idx_of_type[type] (the degree the
 * planner fixed for that type, H2).
 *
 * The space: every (P, mbs, rc, D) of the lists and one (zone, combination) per segment (stage i belongs to segment
 * floor(i * nseg / P), nseg = min(P, seg_max)); the segment digit is zone * n_comb(D) + combination.  Flat index,
 * digits from low to high: seg[nseg-1] .. seg[0], then the positions in d_values, rc_values, mbs_idx; the
 * sub-spaces of the entries of p_values are concatenated.  With granularity 1 and one tensor-parallel degree for
 * all types this is exactly the space of sailor_plan with that degree, index by index. */
#define SAILOR_MIX_UNITS_MAX 16

typedef struct sailor_mixed_space {
    uint32_t n_p, n_mbs, n_rc, n_d, seg_max, granularity;
    uint8_t  p_values[SAILOR_NP_MAX];       /* each 1 .. SAILOR_MIX_P_MAX                                */
    uint8_t  mbs_idx[SAILOR_MBS_MAX];
    uint8_t  rc_values[2];
    uint8_t  tp_idx_of_type[SAILOR_T_MAX];  /* tensor-parallel degree (index) of every GPU type          */
    uint8_t  _pad[6];
    uint16_t d_values[SAILOR_ND_MAX];
} sailor_mixed_space;

typedef struct sailor_mixed_result {
    uint64_t flat;
    double   t_iter;
    double   cost;
    uint64_t peak_mem;
    double   score;
    uint32_t status;
    uint32_t _pad;
    sailor_mixed_plan plan;                 /* stages past P are zero                                    */
} sailor_mixed_result;

/* Number of candidates (host arithmetic).  E_RANGE: a limit above, units(D) beyond SAILOR_MIX_UNITS_MAX, more than
 * 2^63 candidates. */
int sailor_mixed_space_size(const sailor_ctx* ctx, const sailor_mixed_space* s, uint64_t* n_out);

/* Flat index -> plan record (host arithmetic), the inverse of the enumeration order. */
int sailor_mixed_decode(const sailor_ctx* ctx, const sailor_mixed_space* s, uint64_t flat, sailor_mixed_plan* out);

/* Search the whole space: every candidate is built on the device from its flat index, simulated as
 * sailor_simulate_mixed simulates it, classed (the first of invalid, out of memory, over availability, over the
 * budget or under the throughput floor that applies, else feasible) and the k best feasible ones by (score, flat)
 * returned, best first, with their records.  o->flags must be 0 and o->budget_factor_over_cheapest 0 (E_ARG).
 * `topk` is a HOST array of k records; `stats` may be NULL (n_pruned_tp, n_skipped are 0; n_configs counts the
 * (P, mbs, rc, D) tuples).  Uses the availability last set; allocates device memory on first use (grow-only, kept by
 * the context); synchronises the stream.  Errors: E_ARG, E_RANGE (as sailor_mixed_space_size; k > SAILOR_K_MAX),
 * E_NOMEM, E_CUDA, E_DEVICE. */
int sailor_plan_mixed(sailor_ctx* ctx, const sailor_mixed_space* s, const sailor_objective* o, uint32_t k,
                      sailor_mixed_result* topk, uint32_t* n_found, sailor_stats* stats);

/* ---- per-stage GPU types by dynamic programming (Sec. 4.2.2: Eq. 1, T_total, the listing) --------
 *
 * sailor_plan varies the GPU type and zone of at most SAILOR_SEG_MAX segments of a pipeline.  This
 * entry point gives every stage its own GPU type, the way the paper's planner does: by a recursion
 * over the stages that hands stage i its resources, solves stages i+1.. on what is left, and combines
 * the two by T_total.
 *
 * A problem is one configuration (P, mbs, tp, rc, D) of the space (seg_max is ignored) together
 * with one zone order, the order in which zones are filled (the paper's planner loops over region
 * combinations outside the recursion; H5 keeps a stage inside one zone).  All D replicas of a stage
 * use the same GPU type and tp.  A stage goes to the first zone, at or after the previous stage's
 * zone in the order, that still has D*tp GPUs of its type free.  For stage i on type g the
 * recursion tries every type g' for stage i+1 in ascending order, takes the best plan of stages
 * i+1.. for the state that results, and combines (binary64, this order, no fused multiply-add):
 *     t     = (f_i + b_i) + 2 * c(i -> i+1)                 the last stage: f + b
 *     sum   = t + sum_rest          mx = max(t, mx_rest)
 *     sy    = max(sync_i, sy_rest)  up = max(u_i, up_rest)
 *     value = ((sum + N_b * mx) + sy) + up
 * keeping the smallest value (the first among equals).  As in Eq. 1 the rest of the pipeline is
 * the best one for its own state, so the plan found can be worse than the best of all type
 * sequences.  `value` sums the stage times from the last stage backwards; t_iter, cost and
 * peak_mem of a result are the simulator's figures for the written-out plan (stage order), equal
 * to value up to rounding.  The objective is iteration time (o->kind must be MAX_THROUGHPUT, no
 * flags other than SAILOR_DP_FLAG_*, no budget factor).  A budget or a minimum throughput in `o` is checked on the plan the
 * recursion returns for a problem, by the simulator's cost and time (Sec. 4.2: a configuration
 * counts only when it is within the constraint); a problem whose plan fails it drops out.
 *
 * With SAILOR_DP_FLAG_BUDGET_LOOP the budget also steers the recursion, the way Sec. 4.2.3 ("Adding a
 * monetary cost constraint") and the second half of the listing describe.  A stage is charged
 *     C_i = rate_i * (N_b * t_straggler) + C_comm_i
 * (rate_i = (double)(D * tp) * price per second of its GPUs; C_comm_i = (double)(2 * N_b * D * p2p_bytes) * egress
 * of its message to the next stage when that crosses zones) with an ASSUMED straggler: first the stage's own time t.
 * The stages after it are solved with what is left, C_rem = C_cur - C_i (nothing is tried when C_rem <= 0).  If
 * their straggler is not slower than the assumed one, the candidate counts when C_i + their charges <= C_cur; if it
 * is slower, the stage is charged again with that straggler and they are solved again with the smaller remainder.
 * The last stage is its own straggler and counts when its charge is within its limit.  Candidates combine and
 * compare as above.  The remaining budget is an argument of the recursion (a state reached with two different
 * remainders is solved twice), so the tables above do not apply: each problem is walked depth-first by one GPU
 * thread, problems in parallel.  The work can grow as T^P: a branch is cut when what is left cannot pay the
 * cheapest conceivable rest of the pipeline (this changes no result), and a problem that needs more than 2^24 calls
 * of the recursion is given up and counted in n_unfinished.  The charge underestimates the simulator's cost (it
 * leaves out warm-up, cool-down, synchronisation and update time, as the paper's simplification does), so the
 * check of the simulator's cost against the budget still follows, as without the flag.  n_states then counts the
 * calls of the recursion.
 *
 * On the device every problem is a dense table over its states (stage, type, zone position,
 * stages per type already placed in that zone; a type with room for all P stages in a zone is not
 * counted there), filled from the last stage to the first, one launch per stage for all problems
 * of a batch together; batches are cut so that the tables fit `workspace_bytes`. */
/* How sailor_plan_dp lays out and walks its tables, in sailor_objective.flags.  The results do not
 * depend on them; they exist so that every code path can be selected (and tested) through this
 * interface.  Index of a zone position's count vectors: the smaller of the two ways (default), mixed
 * radix whenever it fits (DENSE), by rank whenever it fits (COMPACT).  Threads of a stage's launch: one
 * per reachable count vector for all its types (default), one per reachable count vector and type
 * (BY_TYPE), one per table entry (BY_ENTRY). */
#define SAILOR_DP_FLAG_INDEX_DENSE    0x100u
#define SAILOR_DP_FLAG_INDEX_COMPACT  0x200u
#define SAILOR_DP_FLAG_ENUM_BY_TYPE   0x400u
#define SAILOR_DP_FLAG_ENUM_BY_ENTRY  0x800u
/* Steer the recursion by the budget (Sec. 4.2.3) instead of only checking it on the plan the recursion returns: see
 * sailor_plan_dp.  Needs budget_usd_per_iter > 0; pipelines of at most SAILOR_DP_BUDGET_P_MAX stages. */
#define SAILOR_DP_FLAG_BUDGET_LOOP    0x1000u
#define SAILOR_DP_BUDGET_P_MAX        32

typedef struct sailor_zone_order {
    uint8_t n;                          /* 1 .. SAILOR_Z_MAX zones, each at most once                */
    uint8_t zone[SAILOR_Z_MAX];
    uint8_t _pad[3];
} sailor_zone_order;

typedef struct sailor_dp_result {
    uint32_t config;                    /* configuration index: (((p * n_mbs + mbs) * n_tp + tp) * n_rc + rc) * n_d + d,
                                           positions in the space's lists                             */
    uint32_t order;                     /* index into `orders`                                        */
    double   value;                     /* the recursion's value of the plan                          */
    double   t_iter, cost;              /* the simulator's figures for the plan (Sec. 4.3)            */
    uint64_t peak_mem;
    uint32_t status;                    /* the simulator's status of the plan: 0                      */
    uint8_t  P, mbs_idx, tp_idx, rc;
    uint16_t D;
    uint16_t _pad;
    uint8_t  type[SAILOR_P_MAX];        /* GPU type of every stage                                    */
    uint8_t  zone[SAILOR_P_MAX];        /* zone of every stage                                        */
} sailor_dp_result;

typedef struct sailor_dp_stats {
    uint64_t n_problems;                /* configurations x zone orders                               */
    uint64_t n_solved;                  /* problems that have a plan                                  */
    uint64_t n_over_constraint;         /* of which the plan is over the budget or under the throughput */
    uint64_t n_states;                  /* table entries filled (all problems, all stages)            */
    uint64_t workspace_used;            /* bytes of the largest batch                                 */
    float    kernel_ms;
    uint32_t n_launches, n_batches;
    uint32_t n_unfinished;              /* SAILOR_DP_FLAG_BUDGET_LOOP: problems given up (too many calls)   */
} sailor_dp_stats;

/* Solve every problem of `s` x `orders` and return the k best plans within the constraint by
 * (value, problem index = config * n_orders + order) ascending; *n_found <= k.  `topk` is a HOST array of k records;
 * `stats` may be NULL.  Uses the availability last set.  `workspace_bytes` bounds the device memory
 * of the tables (0 = 8 GiB); it is allocated on first use and kept by the context (grow-only).
 * Errors: E_ARG (null, k == 0, n_orders == 0, a zone twice or out of range, an objective other
 * than plain MAX_THROUGHPUT, the budget loop without a budget), E_RANGE (k >
 * SAILOR_K_MAX, space limits as sailor_plan, a single problem whose tables exceed the workspace or
 * 2^31 entries per stage), E_NOMEM, E_CUDA. */
int sailor_plan_dp(sailor_ctx* ctx, const sailor_space* s, const sailor_zone_order* orders, uint32_t n_orders,
                   const sailor_objective* o, uint64_t workspace_bytes, uint32_t k, sailor_dp_result* topk,
                   uint32_t* n_found, sailor_dp_stats* stats);

/* ---- sustained issue rates of the device (a measurement, not part of the method) -------------------
 *
 * The search is bound by instruction issue, so its throughput is judged against the rate at which
 * the device really issues instructions.  This call times three instruction streams (FP32 fused
 * multiply-add, 32-bit integer multiply-add, FP64 add; eight independent chains per thread, four
 * blocks of 256 threads per SM, about a millisecond each, best of `repeats` runs) with CUDA events on
 * `cuda_stream` and reports warp-instructions per second for each.  It allocates and frees 8 bytes of
 * device memory and synchronises the stream.  Errors: E_ARG (null, repeats == 0), E_CUDA (no context
 * to record the code in: the return value is all there is). */
typedef struct sailor_issue_rates {
    double   ffma_warp_inst_per_s;      /* FP32 pipe stream: what the four schedulers of an SM sustain  */
    double   imad_warp_inst_per_s;      /* integer multiply-add stream                                   */
    double   dadd_warp_inst_per_s;      /* FP64 pipe stream                                              */
    float    ffma_ms, imad_ms, dadd_ms; /* duration of the best run of each stream                       */
    uint32_t sm_count;
    uint64_t warp_inst_per_run;         /* stream instructions one run of a kernel executes              */
} sailor_issue_rates;

int sailor_measure_issue_rates(int cuda_device, void* cuda_stream, uint32_t repeats, sailor_issue_rates* out);

const char* sailor_strerror(int code);
int sailor_last_cuda_error(const sailor_ctx* ctx);   /* cudaError_t of the last E_CUDA      */

#ifdef __cplusplus
}
#endif
#endif /* SAILOR_H */
