// The per-stage recursion under a cost limit (Sailor Sec. 4.2.3, "Adding a monetary cost constraint", and the
// second half of the listing in Sec. 4.2.2).
//
// A stage is charged  C_i = rate_i * (N_b * t_straggler) + C_comm_i  with an ASSUMED straggler: first its own
// time; the stages after it are solved with what is left of the limit, and when their straggler turns out
// slower the stage is charged again with that one and they are solved again, until the assumption holds,
// nothing is left, or they have no plan.  The remaining limit is an argument of the recursion, so a state has no
// single value and the tables of the unlimited search do not apply: every problem (configuration x zone order) is
// walked depth-first by one thread with an explicit stack in global memory.  Problems are independent, which is
// where the parallelism is; a problem's own walk is sequential by nature (each call's limit depends on the
// charges before it).  A branch is cut when what is left cannot pay even the cheapest conceivable rest of the
// pipeline (every later stage alone on its cheapest GPUs, charged for its own compute time): such a branch has no
// plan, so the cut changes nothing but the work.  A problem that would take more than `node_limit` calls is given
// up and reported as unfinished.
#pragma once

#include "sailor_dp.cuh"

namespace sailor {

constexpr uint32_t DP_BUDGET_P_MAX = 32;     // deepest pipeline the limited recursion takes

struct DpbFrame {                    // one call of the recursion: stage `level` on type g at zone position zp
    double limit;                    // what stages level.. may be charged
    double rate, sync, fb, upd;      // of this stage on its GPUs
    double t, comm, assumed, charge; // the candidate being tried: stage time with its message, transfer cost, ...
    double b_sum, b_mx, b_sy, b_up, b_cost;      // best plan of stages level.. so far (b_found)
    uint8_t g, zp, g2, zp2;          // g2: type tried for the next stage, zp2: where first fit puts it
    uint8_t b_found, _pad[3];
    uint8_t u[SAILOR_T_MAX];         // stages per type in zone position zp, this stage included
    uint8_t u2[SAILOR_T_MAX];        // the same for the next stage's position after the move
    uint8_t b_type[DP_BUDGET_P_MAX]; // types of stages level.. of the best plan (indexed by stage)
};

struct DpBudgetParams {
    const unsigned char* blob;
    const uint16_t* avail;
    SpaceDesc sp;
    const DpProblem* problems;
    const double* tabs;
    DpResult* results;               // indexed by problem index
    DpbFrame* frames;                // [n_problems][DP_BUDGET_P_MAX]
    unsigned long long* counters;    // [3] += problems given up, [4] += calls of the recursion
    DpTabLayout lay;
    uint32_t n_problems, T;
    double limit;
    unsigned long long node_limit;
};

__device__ __forceinline__ double dpb_value(double nb, double sum, double mx, double sy, double up) {
    return add_rn(add_rn(add_rn(sum, mul_rn(nb, mx)), sy), up);
}

__global__ void __launch_bounds__(64) dp_budget_kernel(const __grid_constant__ DpBudgetParams bp) {
    const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= bp.n_problems) return;
    const DpProblem& pb = bp.problems[x];
    DpResult& out = bp.results[pb.index];
    out.value = make_inf();
    const uint32_t T = bp.T, P = pb.P;
    const double* tab = bp.tabs + (size_t)pb.config * bp.lay.stride();
    if (*reinterpret_cast<const uint32_t*>(tab + bp.lay.off_nb() + 1) == 0 || P > DP_BUDGET_P_MAX) return;   // no valid plan here
    TabView v;
    v.bind(bp.blob, bp.blob);
    const TabHdr* h = v.h;
    const uint32_t R = h->R, Z = h->Z;
    const uint32_t* okv = reinterpret_cast<const uint32_t*>(tab + bp.lay.off_ok());
    const uint64_t n_b = *reinterpret_cast<const uint64_t*>(tab + bp.lay.off_nb());
    const double nb = (double)n_b;
    const Config k = config_of(bp.sp, pb.config);
    const double gpus = (double)(k.D * h->tp_values[k.tpi]);
    const double xbytes = (double)(2 * n_b * (uint64_t)k.D * v.p2p[k.mi]);
    const double* fbt = tab + bp.lay.off_fb();
    const double* updt = tab + bp.lay.off_upd();
    const double* synct = tab + bp.lay.off_sync();
    const double* c2x = tab + bp.lay.off_c2x();
    DpbFrame* fr = bp.frames + (size_t)x * DP_BUDGET_P_MAX;

    // the least any plan of stages j.. can be charged: every stage alone on the cheapest GPUs it fits, for its own
    // compute time; added up from the last stage backwards, as the recursion adds its charges
    double lb[DP_BUDGET_P_MAX + 1];
    lb[P] = 0.0;
    for (uint32_t j = P; j-- > 0;) {
        double least = make_inf();
        for (uint32_t g = 0; g < T; ++g) {
            if (!((okv[j] >> g) & 1u)) continue;
            for (uint32_t q = 0; q < pb.nz; ++q) {
                const double c = mul_rn(mul_rn(gpus, v.price_s[pb.zone[q] * T + g]), mul_rn(nb, fbt[j * T + g]));
                least = c < least ? c : least;
            }
        }
        lb[j] = add_rn(least, lb[j + 1]);
    }

    unsigned long long nodes = 0;
    bool gave_up = false;
    // result of the call that has just returned
    bool r_found = false;
    double r_sum = 0.0, r_mx = 0.0, r_sy = 0.0, r_up = 0.0, r_cost = 0.0;
    // stage 0: every type, by first fit from the first zone of the order
    bool best_found = false;
    double best_v = make_inf();
    uint8_t best_type[DP_BUDGET_P_MAX];
    for (uint32_t g0 = 0; g0 < T && !gave_up; ++g0) {
        if (!((okv[0] >> g0) & 1u)) continue;
        const uint32_t p0 = pb.cap[0][g0] >= 1 ? 0u : pb.first_later[0][g0];
        if (p0 == DP_NONE) continue;
        if (bp.limit < lb[0]) continue;
        int level = 0;
        {
            DpbFrame& f = fr[0];
            f.g = (uint8_t)g0; f.zp = (uint8_t)p0; f.limit = bp.limit;
            for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) f.u[t] = 0;
            f.u[g0] = 1;
        }
        enum { ENTER, NEXT_TYPE, CHARGE, RESUME } state = ENTER;
        while (level >= 0) {
            DpbFrame& f = fr[level];
            const uint32_t i = (uint32_t)level, g = f.g, z = pb.zone[f.zp], d = z * T + g;
            if (state == ENTER) {
                if (++nodes > bp.node_limit) { gave_up = true; break; }
                f.b_found = 0;
                f.rate = mul_rn(gpus, v.price_s[d]);
                f.sync = synct[i * R + d];
                f.fb = fbt[i * T + g];
                f.upd = updt[i * T + g];
                if (i == P - 1) {                    // the last stage sends nothing and is its own straggler
                    const double charge = mul_rn(f.rate, mul_rn(nb, f.fb));
                    r_found = charge <= f.limit;
                    r_sum = f.fb; r_mx = f.fb; r_sy = f.sync; r_up = f.upd; r_cost = charge;
                    f.b_type[i] = (uint8_t)g;
                    --level;
                    state = RESUME;
                    continue;
                }
                f.g2 = 0;
                state = NEXT_TYPE;
            }
            if (state == NEXT_TYPE) {
                bool placed = false;
                while (f.g2 < T) {
                    const uint32_t g2 = f.g2;
                    if ((okv[i + 1] >> g2) & 1u) {
                        // first fit: this zone while it has room for one more stage of the type, else the next that has
                        uint32_t zp2 = f.zp;
                        if (!(f.u[g2] < pb.cap[f.zp][g2])) zp2 = pb.first_later[f.zp][g2];
                        if (zp2 != DP_NONE) {
                            f.zp2 = (uint8_t)zp2;
                            for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) f.u2[t] = zp2 == f.zp ? f.u[t] : 0;
                            f.u2[g2]++;
                            const uint32_t z2 = pb.zone[zp2], dn = z2 * T + g2;
                            f.t = add_rn(f.fb, c2x[dn * R + d]);
                            f.comm = z2 != z ? mul_rn(xbytes, v.egress[z * Z + z2]) : 0.0;
                            f.assumed = f.t;                 // first: this stage is the straggler
                            placed = true;
                            break;
                        }
                    }
                    ++f.g2;
                }
                if (!placed) {                               // every type tried: hand the best plan back
                    r_found = f.b_found != 0;
                    r_sum = f.b_sum; r_mx = f.b_mx; r_sy = f.b_sy; r_up = f.b_up; r_cost = f.b_cost;
                    --level;
                    state = RESUME;
                    continue;
                }
                state = CHARGE;
            }
            if (state == CHARGE) {
                f.charge = add_rn(mul_rn(f.rate, mul_rn(nb, f.assumed)), f.comm);
                const double rest = f.limit - f.charge;
                if (!(rest > 0.0) || rest < lb[i + 1]) {    // nothing left, or not enough for any rest of the pipeline
                    ++f.g2;
                    state = NEXT_TYPE;
                    continue;
                }
                DpbFrame& c = fr[level + 1];
                c.g = f.g2; c.zp = f.zp2; c.limit = rest;
                for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) c.u[t] = f.u2[t];
                ++level;
                state = ENTER;
                continue;
            }
            // RESUME: the call for stages i + 1.. has returned
            if (!r_found) {
                ++f.g2;
                state = NEXT_TYPE;
                continue;
            }
            if (r_mx <= f.assumed) {                         // the assumption holds
                const double all = add_rn(f.charge, r_cost);
                if (all <= f.limit) {
                    const double c_sum = add_rn(f.t, r_sum), c_mx = dmax(f.t, r_mx), c_sy = dmax(f.sync, r_sy),
                                 c_up = dmax(f.upd, r_up);
                    if (!f.b_found || dpb_value(nb, c_sum, c_mx, c_sy, c_up) < dpb_value(nb, f.b_sum, f.b_mx, f.b_sy, f.b_up)) {
                        f.b_found = 1;
                        f.b_sum = c_sum; f.b_mx = c_mx; f.b_sy = c_sy; f.b_up = c_up; f.b_cost = all;
                        const DpbFrame& c = fr[level + 1];
                        for (uint32_t j = i + 1; j < P; ++j) f.b_type[j] = c.b_type[j];
                        f.b_type[i] = (uint8_t)g;
                    }
                }
                ++f.g2;
                state = NEXT_TYPE;
                continue;
            }
            f.assumed = r_mx;                                // charge again with the straggler that was found
            state = CHARGE;
        }
        if (gave_up) break;
        // the call for stage 0 on g0 has returned (level == -1)
        if (r_found) {
            const double val = dpb_value(nb, r_sum, r_mx, r_sy, r_up);
            if (!best_found || val < best_v) {
                best_found = true;
                best_v = val;
                for (uint32_t j = 0; j < P; ++j) best_type[j] = fr[0].b_type[j];
            }
        }
    }
    atomicAdd(&bp.counters[4], nodes);
    if (gave_up) { atomicAdd(&bp.counters[3], 1ull); return; }
    if (!best_found) return;
    out.value = best_v;
    // zones by first fit, as the recursion placed them; then the plan through the simulator (Sec. 4.3)
    sailor_run runs[DP_BUDGET_P_MAX];
    uint32_t n_runs = 0, zp = 0;
    uint8_t u[SAILOR_T_MAX];
    for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) u[t] = 0;
    for (uint32_t i = 0; i < P; ++i) {
        const uint32_t g = best_type[i];
        uint32_t zp2 = zp;
        if (!(u[g] < pb.cap[zp][g])) zp2 = pb.first_later[zp][g];
        if (zp2 != zp) for (uint32_t t = 0; t < SAILOR_T_MAX; ++t) u[t] = 0;
        u[g]++;
        zp = zp2;
        const uint8_t z = pb.zone[zp];
        out.type[i] = (uint8_t)g;
        out.zone[i] = z;
        if (n_runs && runs[n_runs - 1].type == g && runs[n_runs - 1].zone == z) runs[n_runs - 1].n_stages++;
        else {
            runs[n_runs].type = (uint8_t)g; runs[n_runs].zone = z;
            runs[n_runs].tp_idx = (uint8_t)k.tpi; runs[n_runs].n_stages = 1;
            ++n_runs;
        }
    }
    uint32_t cnt[R_MAX];
    const SimOut so = simulate_runs(v, bp.avail, P, n_runs, k.D, k.mi, k.rc, runs, DP_BUDGET_P_MAX, cnt, 1);
    out.t_iter = so.t_iter;
    out.cost = so.cost;
    out.peak_mem = so.peak_mem;
    out.status = so.status;
}

}  // namespace sailor
