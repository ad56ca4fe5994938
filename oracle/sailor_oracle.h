/*
 * sailor_oracle.h — TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded CPU statement of what the Sailor plan simulator and the
 * exhaustive plan search compute (Sailor, SOSP'25: Sec. 4.2 planner overview and H1-H5,
 * Sec. 4.2.2 T_total, Sec. 4.2.3 cost constraint, Sec. 4.3 simulator).  It exists to check the
 * CUDA library; it shares no source, header, table or helper with it and nothing in the
 * product may call it.  Every stage of every plan is walked layer by layer; nothing is
 * cached, blocked, fused or reordered.
 *
 * Pins (see tests, all run without a GPU): three hand-computed two-stage cases and one
 * hand-computed three-stage case with embedding/head layers, recomputation, alpha > 0 and
 * mixed tensor parallelism; two hand-computed cases with fitted bandwidth polynomials (boundary
 * link and all-reduce); the homogeneous closed form (P + N_b) * t; monotonicity and
 * scaling invariants; an independent nested-loop enumeration and brute-force minimum on
 * tiny clusters.  The pruned search modes (H2-H4): three hand-worked searches, equality with the
 * exhaustive search when no mode is on, and a brute-force restatement over per-candidate results
 * on tiny clusters (group minimum over tensor-parallel degrees, per-configuration bests).  The
 * dynamic-programming recursion and the simulator for plans that mix GPU types inside a stage: see the
 * comments above their declarations below.
 * Parity unpinned: the absolute realism of the outputs against real clusters (Sec. 5.1
 * reports 4-6 % error on hardware this repository cannot reach).
 */
#ifndef SAILOR_ORACLE_H
#define SAILOR_ORACLE_H

#include <stdint.h>

#define ORC_KINDS 3            /* 0 embedding, 1 transformer block, 2 head */
#define ORC_STAGES_MAX 128
#define ORC_SEG_MAX 8

/* status bits */
#define ORC_INVALID 1u
#define ORC_OVER_AVAIL 2u
#define ORC_OOM 4u

/* objective kinds: what is minimised */
#define ORC_OBJ_TIME 0           /* maximise throughput            */
#define ORC_OBJ_COST 1           /* minimise cost per iteration    */
#define ORC_OBJ_TIME_X_COST 2    /* maximise throughput per dollar */

typedef struct orc_inputs {
    /* training job */
    uint32_t n_blocks, has_embed, has_head, heads;
    uint64_t gbs;
    uint32_t mul_factor, dtype_size, grad_dtype_size;
    /* table shapes */
    uint32_t n_types, n_zones, n_tp, n_mbs;
    const uint32_t* tp_values;     /* [n_tp]  */
    const uint32_t* mbs_values;    /* [n_mbs] */
    /* per-layer profile, Sec. 4.1 */
    const double* fwd;             /* [kind][type][tp][mbs] */
    const double* bwd;             /* [kind][type][tp][mbs] */
    const double* upd;             /* [kind][type][tp]      */
    const uint64_t* params;        /* [kind]                */
    const uint64_t* act_saved;     /* [kind][tp][mbs]       */
    const uint64_t* act_ckpt;      /* [kind][tp][mbs]       */
    const uint64_t* act_work;      /* [kind][tp][mbs]       */
    const uint64_t* p2p_bytes;     /* [mbs]                 */
    /* cluster */
    const uint64_t* capacity;      /* [type] */
    const uint64_t* reserved;      /* [type] */
    const uint32_t* gpus_per_node; /* [type] */
    const double* price_per_hour;  /* [zone][type] */
    const double* intra_alpha;     /* [zone][type] */
    const double* intra_inv_bw;
    const double* inter_alpha;
    const double* inter_inv_bw;
    const double* zone_alpha;      /* [zone][zone] */
    const double* zone_inv_bw;
    const double* egress;          /* [zone][zone] dollars per byte */
    /* optional fitted bandwidth polynomials, Sec. 4.1: bandwidth(m) = p0 + p1 m + p2 m^2 + p3 m^3 bytes/s
     * for a message of m bytes; NULL = the link uses inv_bw */
    const double* intra_bw_poly;   /* [zone][type][4] or NULL */
    const double* inter_bw_poly;   /* [zone][type][4] or NULL */
    const double* zone_bw_poly;    /* [zone][zone][4] or NULL */
    const uint16_t* avail;         /* [zone][type] */
} orc_inputs;

/* a plan with every stage written out */
typedef struct orc_plan {
    uint32_t P, mbs_idx, rc, D;
    uint32_t type[ORC_STAGES_MAX];
    uint32_t zone[ORC_STAGES_MAX];
    uint32_t tp_idx[ORC_STAGES_MAX];
} orc_plan;

typedef struct orc_out {
    uint32_t status;
    uint32_t _pad;
    double t_iter;
    double cost;
    uint64_t peak_mem;
    /* intermediate quantities, for the hand-computed pins */
    double t_pp, t_sync, t_update, rate_per_s, c_comm;
    uint64_t n_b;
    uint64_t stage_mem[ORC_STAGES_MAX];
    double stage_t[ORC_STAGES_MAX];
    double stage_c[ORC_STAGES_MAX];
    double stage_sync[ORC_STAGES_MAX];
} orc_out;

typedef struct orc_space {
    uint32_t n_p, n_mbs, n_tp, n_rc, n_d, seg_max;
    const uint32_t* p_values;
    const uint32_t* mbs_idx;
    const uint32_t* tp_idx;
    const uint32_t* rc_values;
    const uint32_t* d_values;
} orc_space;

typedef struct orc_objective {
    uint32_t kind;
    uint32_t _pad;
    double budget;        /* dollars per iteration, <= 0: none */
    double min_rate;      /* iterations per second, <= 0: none */
} orc_objective;

typedef struct orc_hit {
    uint64_t flat;
    double score, t_iter, cost;
    uint64_t peak_mem;
} orc_hit;

typedef struct orc_counts {
    uint64_t n_total, n_invalid, n_oom, n_over_avail, n_over_constraint, n_feasible;
    double min_cost;      /* smallest cost among the feasible plans, 0 if there is none */
} orc_counts;

void orc_simulate(const orc_inputs* in, const orc_plan* plan, orc_out* out);
uint64_t orc_space_size(const orc_inputs* in, const orc_space* sp);
int orc_decode(const orc_inputs* in, const orc_space* sp, uint64_t flat, orc_plan* plan);
/* walk flat indices lo <= flat < hi in steps of `stride`; keep the k best feasible plans in
 * (score, flat) ascending order; returns how many were kept */
uint32_t orc_search(const orc_inputs* in, const orc_space* sp, const orc_objective* obj,
                    uint64_t lo, uint64_t hi, uint64_t stride, uint32_t k, orc_hit* hits,
                    orc_counts* counts);
/* simulate chosen flat indices: out arrays of n */
void orc_simulate_flat(const orc_inputs* in, const orc_space* sp, const uint64_t* flat, uint64_t n,
                       uint32_t* status, double* t_iter, double* cost, uint64_t* peak_mem);
/* simulate n written-out plans */
void orc_simulate_batch(const orc_inputs* in, const orc_plan* plans, uint64_t n,
                        uint32_t* status, double* t_iter, double* cost, uint64_t* peak_mem);

/* ---- pruning heuristics of the planner as search modes (Sec. 4.2.1) ----------------------------
 *
 * ORC_PRUNE_D_ORDER (H3, H4).  A group is everything of a configuration but its data-parallel degree:
 * (P, mbs, tp, recomputation).  Inside a group the degrees of the space are tried from the largest
 * down when throughput is maximised (H3) and from the smallest up when cost is minimised (H4).
 * Degrees that have no feasible plan are passed over until the first feasible one (H3 starts from the
 * largest degree the available GPUs allow, H4 raises the degree until the constraint is met); after that
 * the next degree is tried only while the best objective value of the group's last degree was strictly better
 * than that of the degree before it.  The degree at which the improvement stops has been evaluated
 * and its plans compete for the top-k like all others; the remaining degrees are never looked at.
 * The paper states the rule for the two objectives only: any other objective is an error (-1).
 *
 * ORC_PRUNE_MIN_TP (H2, extended).  H2 as printed drops tensor-parallel degrees below the minimum that
 * fits in memory, which the memory check already does.  The mode goes one step further and keeps,
 * of the plans that differ only in the (plan-wide) tensor-parallel degree, only the one with the
 * smallest degree that is valid and fits: a plan is dropped when some smaller degree of the space's
 * list gives a valid plan in which every stage fits.  Dropped plans are counted in n_pruned_tp, after
 * the invalid and out-of-memory classes and before the availability check.
 */
#define ORC_PRUNE_D_ORDER 1u
#define ORC_PRUNE_MIN_TP 2u

typedef struct orc_pruned_counts {
    orc_counts looked_at;        /* classes over the candidates of the evaluated configurations;
                                    n_total also contains n_pruned_tp */
    uint64_t n_pruned_tp;
    uint64_t n_skipped;          /* candidates of configurations that early termination never reached */
    uint64_t n_configs, n_configs_evaluated;
} orc_pruned_counts;

/* whole space; returns the number of hits kept (<= k) or -1 for an unsupported request */
int32_t orc_search_pruned(const orc_inputs* in, const orc_space* sp, const orc_objective* obj, uint32_t modes,
                          uint32_t k, orc_hit* hits, orc_pruned_counts* counts);


/* ---- per-stage resource assignment by dynamic programming (Sec. 4.2.2: Eq. 1, T_total, the listing) ----
 *
 * A problem fixes P, mbs, tp, recomputation, D and the order in which zones are filled (the paper's
 * planner loops over region combinations outside the recursion).  The recursion chooses the GPU type of
 * each stage (all D replicas of a stage alike); a stage goes to the first zone, at or after the
 * previous stage's zone in the order, with D*tp GPUs of its type free.  For stage i on type g it tries
 * every type g' for stage i+1 in ascending order, solves stages i+1.. for what is left (remembered per
 * state: stage, type, zone position, stages per type already placed in that zone), and combines:
 *     t     = (f_i + b_i) + 2 * c(i -> i+1)            [the last stage: f + b]
 *     sum   = t + sum_rest        mx = max(t, mx_rest)
 *     sy    = max(sync_i, sy_rest)        up = max(u_i, up_rest)
 *     value = ((sum + N_b * mx) + sy) + up              [T_total of Sec. 4.2.2 plus the update of Sec. 4.3]
 * keeping the smallest value (the first found among equals).  The rest of the pipeline is always the best
 * one for its own state, as in Eq. 1, so the result can be worse than the true optimum over all type
 * sequences.  Pins: equality with a plain recursion without the memory; a hand-worked case in which the
 * recursion provably misses the optimum by a known amount; brute force over all type sequences (never
 * better than the optimum, equal for P <= 2, the plan obeys first fit and availability, and the
 * simulator reproduces the value from the plan).  The budget loop of Sec. 4.2.3 is not part of it. */
#define ORC_DP_T_MAX 8

typedef struct orc_dp_problem {
    uint32_t P, mbs_idx, tp_idx, rc, D;
    uint32_t n_zones_used;
    uint32_t zone_list[16];      /* zones in the order they are filled */
} orc_dp_problem;

typedef struct orc_dp_result {
    int32_t found;               /* 0: no plan fits */
    uint32_t _pad;
    double value;                /* the recursion's own value of the kept plan (sums run from the last stage) */
    uint64_t n_states;           /* states solved (not counting remembered ones) */
    orc_plan plan;
} orc_dp_result;

/* returns 0, or -1 for sizes beyond the limits; use_memo = 0 is the plain recursion */
int orc_solve_dp(const orc_inputs* in, const orc_dp_problem* pb, int use_memo, orc_dp_result* out);

/* The same recursion under a cost limit (Sec. 4.2.3, "Adding a monetary cost constraint", and the second half of
 * the listing).  A stage is charged by the simplified cost of that section:
 *     C_i = rate_i * (N_b * t_straggler) + C_comm_i
 * rate_i = (double)(D * tp) * (price_per_hour / 3600) of its GPUs, C_comm_i = the transfer cost of its message
 * to the next stage when that crosses zones ((double)(2 * N_b * D * p2p_bytes) * egress), and t_straggler the
 * ASSUMED straggler: first the stage's own time; the stages after it are solved with what is left of the limit,
 * C_rem = C_cur - C_i; when their straggler turns out slower than the assumed one, the stage is charged again
 * with that straggler and they are solved again with the smaller remainder, until the assumption holds
 * (their straggler <= the assumed one: then the plan counts if C_i + their cost <= C_cur), nothing is left
 * (C_rem <= 0) or they have no plan.  The last stage is its own straggler and counts if its charge is within
 * its limit.  Candidates combine and compare exactly as in orc_solve_dp.  The remaining limit is an argument of
 * the recursion, so nothing is remembered between calls here (a state reached with two different remainders is
 * solved twice); with limit = +infinity the result is orc_solve_dp's bit for bit.
 * charged_cost is the sum of the charges of the kept plan; n_states counts the calls of the recursion. */
typedef struct orc_dp_budget_result {
    int32_t found;
    uint32_t _pad;
    double value;
    double charged_cost;
    uint64_t n_states;
    orc_plan plan;
} orc_dp_budget_result;

int orc_solve_dp_budget(const orc_inputs* in, const orc_dp_problem* pb, double limit, orc_dp_budget_result* out);


/* ---- plans whose stages mix GPU types among their replicas ------------------------------------------
 *
 * The paper's plan gives every stage D replicas, each with its own (GPU type, tp), all in one zone
 * (Sec. 4.2 problem statement, H1, H5), and its framework runs such plans (Sec. 4.4).  Here a stage lists
 * its replicas as groups of `count` equal replicas.  What the paper leaves open is read as follows:
 *   - replicas are numbered group after group; pipeline k is replica k of every stage; every pipeline
 *     processes N_b = gbs / (D * mbs) microbatches; T_pp of a pipeline is sum_i t_i + N_b * max_i t_i over its
 *     own stages, and T_iter = max_k T_pp(k) + T_sync + T_update (Sec. 4.3);
 *   - the message between two neighbouring replicas stays inside a node only when they have the same GPU
 *     type and the two groups they belong to fit one node together; across zones the zone link; otherwise
 *     the slower of the two types' inter-node links (as for plans without mixing);
 *   - a stage's all-reduce moves the largest gradient shard among its groups (smallest tp); a single group
 *     that fits a node uses the intra-node link, otherwise the ring is as slow as the slowest group's
 *     inter-node link;
 *   - memory is checked per group (stage, tp, GPU type); T_update and the price rate run over all groups.
 * A plan whose stages all have one group is the plan of orc_simulate and gives bit-identical results
 * (pinned), and a plan whose stages all split D the same way has exactly the slower of its two
 * homogeneous pipelines (pinned against orc_simulate); one case is worked by hand. */
#define ORC_GROUPS_MAX 4

typedef struct orc_replica_group { uint32_t type, tp_idx, count; } orc_replica_group;
typedef struct orc_mixed_stage { uint32_t zone, n_groups; orc_replica_group group[ORC_GROUPS_MAX]; } orc_mixed_stage;
typedef struct orc_mixed_plan {
    uint32_t P, mbs_idx, rc, D;
    orc_mixed_stage stage[ORC_STAGES_MAX];
} orc_mixed_plan;

void orc_simulate_mixed(const orc_inputs* in, const orc_mixed_plan* plan, orc_out* out);
void orc_simulate_mixed_batch(const orc_inputs* in, const orc_mixed_plan* plans, uint64_t n, uint32_t* status,
                              double* t_iter, double* cost, uint64_t* peak_mem);

/* ---- searching over such plans (Sec. 4.2.2 "Implementation": the planner generates, per stage, the resource
 * combinations of different GPU types that give the stage its D replicas) --------------------------------------
 *
 * A combination splits the D replicas of a stage over the GPU types: n_g replicas on type g, sum = D.  To keep
 * the number of combinations bounded the split is made in `granularity` equal parts when granularity divides D
 * (a part = D / granularity replicas), else replica by replica: units(D) = granularity or D, and a combination is a
 * tuple (u_0 .. u_{T-1}) of non-negative units that add up to units(D), at most ORC_GROUPS_MAX of them non-zero;
 * combinations are numbered in DESCENDING lexicographic order of the tuple (everything on type 0 first; with one
 * unit, combination c is "everything on type c").  A stage built from a combination lists
 * its non-empty types in ascending order (group q = the q-th such type, count = units * D / units(D), tensor
 * parallel degree tp_idx_of_type[type]: the degree the planner fixed for that type, H2).
 *
 * Space: as orc_space, but without the tensor-parallel list (it is per type) and with a (zone, combination) per
 * segment instead of a (zone, type): stage i belongs to segment floor(i * nseg / P), nseg = min(P, seg_max <= 4); the
 * segment digit is zone * n_comb(D) + combination.  Flat index, low to high: seg[nseg-1] .. seg[0]; then the
 * positions in d_values, rc_values, mbs_idx; the sub-spaces of p_values concatenated.  The radix of a segment digit
 * depends on D. */
typedef struct orc_mixed_space {
    uint32_t n_p, n_mbs, n_rc, n_d, seg_max, granularity;
    const uint32_t *p_values, *mbs_idx, *rc_values, *d_values;
    const uint32_t* tp_idx_of_type;      /* [n_types] */
} orc_mixed_space;

/* number of combinations for a degree, and the c-th one (units per type); -1 if c is out of range */
uint64_t orc_mixed_n_comb(const orc_inputs* in, const orc_mixed_space* sp, uint32_t D);
int orc_mixed_comb(const orc_inputs* in, const orc_mixed_space* sp, uint32_t D, uint64_t c, uint32_t* units_per_type);

uint64_t orc_mixed_space_size(const orc_inputs* in, const orc_mixed_space* sp);
int orc_mixed_decode(const orc_inputs* in, const orc_mixed_space* sp, uint64_t flat, orc_mixed_plan* out);

/* every candidate of [lo, hi) simulated, classified (first of invalid, oom, over availability, over the constraint
 * that applies, else feasible) and the k best by (score, flat) kept: as orc_search */
uint32_t orc_search_mixed(const orc_inputs* in, const orc_mixed_space* sp, const orc_objective* obj, uint64_t lo,
                          uint64_t hi, uint32_t k, orc_hit* hits, orc_counts* counts);

#endif
