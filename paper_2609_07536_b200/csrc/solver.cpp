// Launch-time analytical selector of the communication-CTA count (host only).
//
// Section III-D, Algorithm 1: for every legal C evaluate the wave-quantized makespan
//   R(C) = ceil(C / o_comm)                      (Eq. 1)
//   P(C) = o_comp floor((G - R(C)) / slot_sms)   (Eq. 3; slot_sms = SMs per compute slot)
//   A_s  = ceil((s+1) W_comp / P)                (Eq. 9)
//   q    = rho ceil(W_comm / C)                  (Eq. 8, Eq. 10)
//   F_s  = max(A_s, F_{s-1}) + q,  T = F_{L-1}   (Eq. 11, Eq. 12)
// and keep the lexicographic minimum of (T, Delta_comp, C), Delta_comp = V_comp P - W_comp
// (tie breaker).  rho is carried in fixed point (2^-20) so that "the same T(C)" is an exact
// integer comparison.  No CUDA call, no allocation, no global state.

#include <chrono>
#include <cstdint>

#include "../../include/moe_b200.h"

namespace {

constexpr int kRhoShift = 20;

inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline uint32_t ceil_div32(uint32_t a, uint32_t b) { return (a + b - 1) / b; }

struct Candidate {
    int64_t T_q;
    int64_t delta;
    int32_t C, R, P;
};

// One candidate.  32-bit divisions when every dividend fits (the common case), else 64-bit.
inline bool evaluate(int32_t C, int64_t Wc, int64_t Wm, int32_t L, int32_t G, int32_t o_comp,
                     int32_t o_comm, int32_t slot_sms, int64_t rho_q, bool small, bool drain_help, Candidate *out)
{
    const int32_t R = (C + o_comm - 1) / o_comm;
    // Eq. 3, with a compute slot that may span several SMs (a CTA pair): only whole slots count
    const int64_t P = G > R ? (int64_t)o_comp * ((G - R) / slot_sms) : 0;
    if (P <= 0) return false;
    int64_t F = 0;
    int64_t V_comp;
    if (drain_help) {
        // Extension (not in the paper): once the last compute wave is over, the compute CTAs serve
        // communication tiles too.  Splits 0..L-2 follow Eq. 11; the tiles still queued at A_{L-1}
        // (whole waves of C) plus the last split's W_comm are served by C + H workers, H = the CTAs
        // that were computing.
        int64_t v_comm, A_last;
        if (small) {
            const uint32_t p = (uint32_t)P, wc = (uint32_t)Wc;
            v_comm = ceil_div32((uint32_t)Wm, (uint32_t)C);
            const int64_t q = rho_q * v_comm;
            uint32_t num = 0, a0 = 0;
            for (int32_t s = 0; s + 1 < L; ++s) {
                num += wc;
                const uint32_t a = ceil_div32(num, p);
                if (s == 0) a0 = a;
                const int64_t A = (int64_t)a << kRhoShift;
                F = (A > F ? A : F) + q;
            }
            const uint32_t al = ceil_div32(num + wc, p);
            A_last = (int64_t)al << kRhoShift;
            V_comp = (L > 1) ? a0 : al;
        } else {
            v_comm = ceil_div64(Wm, C);
            const int64_t q = rho_q * v_comm;
            for (int32_t s = 0; s + 1 < L; ++s) {
                const int64_t A = ceil_div64((int64_t)(s + 1) * Wc, P) << kRhoShift;
                F = (A > F ? A : F) + q;
            }
            A_last = ceil_div64((int64_t)L * Wc, P) << kRhoShift;
            V_comp = ceil_div64(Wc, P);
        }
        int64_t backlog = 0;
        if (F > A_last && rho_q > 0) {
            // ceil((F - A_last) / rho_q): quotient from a double division, then made exact
            const int64_t num = F - A_last;
            int64_t w = (int64_t)((double)num / (double)rho_q);
            while (w * rho_q < num) ++w;
            while (w > 0 && (w - 1) * rho_q >= num) --w;
            backlog = w * C;
            if (backlog > (int64_t)(L - 1) * Wm) backlog = (int64_t)(L - 1) * Wm;
        }
        const int64_t workers = (int64_t)C + P * slot_sms / o_comp;
        const int64_t rem = backlog + Wm;
        const int64_t waves = (small && workers < 0x7FFFFFFF) ? (int64_t)ceil_div32((uint32_t)rem, (uint32_t)workers)
                                                              : ceil_div64(rem, workers);
        F = A_last + rho_q * waves;
    } else if (small) {
        const uint32_t p = (uint32_t)P, wc = (uint32_t)Wc;
        const uint32_t v_comm = ceil_div32((uint32_t)Wm, (uint32_t)C);
        const int64_t q = rho_q * (int64_t)v_comm;
        uint32_t num = 0;
        uint32_t a0 = 0;
        for (int32_t s = 0; s < L; ++s) {
            num += wc;
            const uint32_t a = ceil_div32(num, p);
            if (s == 0) a0 = a;
            const int64_t A = (int64_t)a << kRhoShift;
            F = (A > F ? A : F) + q;
        }
        V_comp = a0;
    } else {
        const int64_t v_comm = ceil_div64(Wm, C);
        const int64_t q = rho_q * v_comm;
        for (int32_t s = 0; s < L; ++s) {
            const int64_t A = ceil_div64((int64_t)(s + 1) * Wc, P) << kRhoShift;
            F = (A > F ? A : F) + q;
        }
        V_comp = ceil_div64(Wc, P);
    }
    out->T_q = F;
    out->delta = V_comp * P - Wc;
    out->C = C;
    out->R = R;
    out->P = (int32_t)P;
    return true;
}

}  // namespace

extern "C" int32_t plan_partition(const int32_t *routed_tile_counts, int32_t n_experts,
                                  const moe_occupancy *occ, const moe_sm_limits *limits,
                                  const moe_shape *shape, const moe_rho *rho, moe_plan *out)
{
    if (!routed_tile_counts || !occ || !limits || !shape || !rho || !out) return MOE_ERR_NULL;
    if (n_experts < 0 || shape->T < 0 || shape->H < 1 || shape->L < 1 || shape->L > MOE_MAX_L ||
        shape->EP < 1 || shape->TP < 1 || shape->I < 1 || shape->k_tot < 1 ||
        occ->tile_m < 1 || occ->tile_n < 1 || occ->comm_tile_m < 1 || occ->comm_tile_n < 1 ||
        occ->o_comp < 1 || occ->o_comm < 1 || occ->comp_slot_sms < 1 || limits->G < 1)
        return MOE_ERR_SHAPE;

    // Eq. 16: sum of the routed tile counts; Eq. 5: compute tiles per split (g = TP groups).
    int64_t S = 0;
    for (int32_t e = 0; e < n_experts; ++e) {
        if (routed_tile_counts[e] < 0) return MOE_ERR_SHAPE;
        S += routed_tile_counts[e];
    }
    const int64_t split_w = ceil_div64(shape->H, shape->L);
    const int64_t Wc = (int64_t)shape->TP * S * ceil_div64(split_w, occ->tile_n);

    // Eq. 7 summed over the emulated ranks: rank d owns a contiguous block of ceil(T/EP) tokens.
    const int64_t blk = ceil_div64(shape->T, shape->EP);
    int64_t tok_tiles = 0;
    for (int32_t d = 0; d < shape->EP; ++d) {
        int64_t own = shape->T - (int64_t)d * blk;
        if (own > blk) own = blk;
        if (own > 0) tok_tiles += ceil_div64(own, occ->comm_tile_m);
    }
    const int64_t Wm = tok_tiles * ceil_div64(split_w, occ->comm_tile_n);
    if (Wc > INT32_MAX || Wm > INT32_MAX) return MOE_ERR_SHAPE;

    // Eq. 14 (one product over one product; integer factors are exact in double).
    const int64_t K = shape->I / shape->TP;
    if (K < 1 || rho->K_ref < 1 || rho->tile_m_ref < 1 || rho->tile_n_ref < 1) return MOE_ERR_SHAPE;
    double num, den;
    if (rho->mode == MOE_RHO_PAPER) {
        if (rho->D_ref < 1) return MOE_ERR_SHAPE;
        num = (double)((int64_t)rho->K_ref * rho->tile_m_ref * rho->tile_n_ref * shape->EP);
        den = (double)(K * occ->tile_m * occ->tile_n * rho->D_ref);
    } else if (rho->mode == MOE_RHO_LOCAL) {
        if (rho->rows_ref < 1 || rho->comm_cols_ref < 1) return MOE_ERR_SHAPE;
        const int64_t rows = (int64_t)shape->k_tot * shape->TP + 1;
        const int64_t cols = split_w < occ->comm_tile_n ? split_w : occ->comm_tile_n;
        num = (double)((int64_t)rho->K_ref * rho->tile_m_ref * rho->tile_n_ref * rows * cols);
        den = (double)(K * occ->tile_m * occ->tile_n * rho->rows_ref * rho->comm_cols_ref);
    } else {
        return MOE_ERR_SHAPE;
    }
    const double rho_v = rho->rho_ref * num / den;
    if (!(rho_v >= 0.0) || rho_v > 1.0e9) return MOE_ERR_SHAPE;
    const double scaled = rho_v * (double)(1 << kRhoShift) + 0.5;
    const int64_t rho_q = (int64_t)scaled;  // scaled >= 0.5: truncation is floor

    const int32_t L = shape->L, G = limits->G, o_comp = occ->o_comp, o_comm = occ->o_comm, slot = occ->comp_slot_sms;
    const bool small = (int64_t)L * Wc < (int64_t)0x7FFFFF00 && Wm < (int64_t)0x7FFFFF00 &&
                       (int64_t)o_comp * G < (int64_t)0x7FFFFF00;

    Candidate best{};
    bool have = false;
    const bool dh = limits->drain_help != 0;
    if (limits->force_comm_ctas > 0 || limits->selector_off) {
        const int32_t C = limits->force_comm_ctas > 0 ? limits->force_comm_ctas : limits->default_C;
        if (C < 1) return MOE_ERR_PLAN_INFEASIBLE;
        have = evaluate(C, Wc, Wm, L, G, o_comp, o_comm, slot, rho_q, small, dh, &best);
    } else if (!small) {
        for (int32_t C = 1; C <= limits->C_max; ++C) {
            Candidate c;
            if (!evaluate(C, Wc, Wm, L, G, o_comp, o_comm, slot, rho_q, small, dh, &c)) break;  // P only falls
            if (!have || c.T_q < best.T_q || (c.T_q == best.T_q && c.delta < best.delta)) {
                best = c;
                have = true;
            }
        }
    } else {
        // Algorithm 1 over C = 1..C_max without a division in the loop: as C grows, P(C) only falls and
        // ceil(W_comm / C) only falls, so every ceiling is carried from the previous candidate and moved
        // to its new exact value with a few multiply-compare steps (same integers as the plain formulas).
        int64_t qa[MOE_MAX_L];           // qa[s] = ceil((s+1) W_comp / P)
        for (int32_t s = 0; s < L; ++s) qa[s] = 0;
        int64_t v = Wm;                  // ceil(W_comm / C), C = 1
        int64_t P_prev = 0;
        const double inv_rho = rho_q > 0 ? 1.0 / (double)rho_q : 0.0;
        for (int32_t C = 1; C <= limits->C_max; ++C) {
            const int32_t R = (o_comm == 1) ? C : (C + o_comm - 1) / o_comm;
            if (G <= R) break;
            const int64_t P = (slot == 1) ? (int64_t)o_comp * (G - R) : (int64_t)o_comp * ((G - R) / slot);
            if (P <= 0) break;
            if (P != P_prev) {
                if (P_prev == 0) {
                    for (int32_t s = 0; s < L; ++s) qa[s] = ceil_div64((int64_t)(s + 1) * Wc, P);
                } else {
                    for (int32_t s = 0; s < L; ++s) {
                        const int64_t num = (int64_t)(s + 1) * Wc;
                        int64_t q = qa[s];
                        while (q * P < num) ++q;
                        qa[s] = q;
                    }
                }
                P_prev = P;
            }
            while (v > 1 && (v - 1) * C >= Wm) --v;
            const int64_t qc = rho_q * v;
            int64_t F = 0;
            if (!dh) {
                for (int32_t s = 0; s < L; ++s) {                       // Eq. 11
                    const int64_t A = qa[s] << kRhoShift;
                    F = (A > F ? A : F) + qc;
                }
            } else {
                for (int32_t s = 0; s + 1 < L; ++s) {
                    const int64_t A = qa[s] << kRhoShift;
                    F = (A > F ? A : F) + qc;
                }
                const int64_t A_last = qa[L - 1] << kRhoShift;
                int64_t backlog = 0;
                if (F > A_last && rho_q > 0) {
                    const int64_t num = F - A_last;
                    int64_t w = (int64_t)((double)num * inv_rho);
                    while (w * rho_q < num) ++w;
                    while (w > 0 && (w - 1) * rho_q >= num) --w;
                    backlog = w * C;
                    if (backlog > (int64_t)(L - 1) * Wm) backlog = (int64_t)(L - 1) * Wm;
                }
                const int64_t workers = (int64_t)C + P * slot / o_comp;
                const int64_t rem = backlog + Wm;
                int64_t waves = rem > 0 ? 1 : 0;
                if (rem > 8 * workers) waves = ceil_div64(rem, workers);
                else while (waves * workers < rem) ++waves;
                F = A_last + rho_q * waves;
            }
            const int64_t delta = qa[0] * P - Wc;                        // tie breaker, V_comp = qa[0]
            // ascending C: a strict improvement of (T, Delta) is needed to replace the incumbent
            if (!have || F < best.T_q || (F == best.T_q && delta < best.delta)) {
                best.T_q = F;
                best.delta = delta;
                best.C = C;
                best.R = R;
                best.P = (int32_t)P;
                have = true;
            }
        }
    }
    if (!have) return MOE_ERR_PLAN_INFEASIBLE;

    out->comm_ctas = best.C;
    out->R = best.R;
    out->P = best.P;
    out->W_comp = (int32_t)Wc;
    out->W_comm = (int32_t)Wm;
    out->delta = (int32_t)best.delta;
    out->pred_T_q = best.T_q;
    out->rho_q = rho_q;
    out->mode = MOE_MODE_FUSED;
    out->debug_withhold_tile = -1;
    out->drain_help = limits->drain_help != 0 ? 1 : 0;
    out->co_warps = 0;
    if (limits->drain_help != 0 && limits->co_warps_max > 0 && limits->force_co_warps > 0)
        out->co_warps = limits->force_co_warps < limits->co_warps_max ? limits->force_co_warps : limits->co_warps_max;
    return MOE_OK;
}

// Mean cost of one plan_partition() call in nanoseconds (steady_clock), over `iters` calls that
// rotate through `n_sets` routed-count vectors laid out back to back.  Measurement aid for the
// solver-overhead figure of Section IV-B; returns the sum of the chosen C values through
// `checksum` so that the calls cannot be optimised away.
extern "C" int32_t moe_time_plan_partition(const int32_t *routed_tile_counts, int32_t n_sets,
                                           int32_t n_experts, const moe_occupancy *occ,
                                           const moe_sm_limits *limits, const moe_shape *shape,
                                           const moe_rho *rho, int64_t iters, double *mean_ns,
                                           int64_t *checksum)
{
    if (!routed_tile_counts || !mean_ns || n_sets < 1 || iters < 1) return MOE_ERR_NULL;
    moe_plan plan;
    int64_t sum = 0;
    int32_t rc = MOE_OK;
    const auto t0 = std::chrono::steady_clock::now();
    int32_t set = 0;
    for (int64_t i = 0; i < iters; ++i) {
        rc = plan_partition(routed_tile_counts + (size_t)set * n_experts, n_experts, occ, limits, shape, rho, &plan);
        if (rc != MOE_OK) break;
        sum += plan.comm_ctas;
        if (++set == n_sets) set = 0;
    }
    const auto t1 = std::chrono::steady_clock::now();
    *mean_ns = std::chrono::duration<double, std::nano>(t1 - t0).count() / (double)iters;
    if (checksum) *checksum = sum;
    return rc;
}

// Section III-E: when the routed counts exist only on the device, the selector runs on a
// normalised-load estimate instead of paying a device-to-host copy and a synchronisation for scheduling
// alone.  The estimate spreads the R = T * k_tot assignments evenly over the E_tot experts:
// every expert gets ceil(R / E_tot) rows, i.e. ceil(ceil(R / E_tot) / T_M) tiles (Eq. 16 on those counts).
extern "C" int32_t plan_partition_estimate(const moe_occupancy *occ, const moe_sm_limits *limits,
                                           const moe_shape *shape, const moe_rho *rho, moe_plan *out)
{
    if (!occ || !limits || !shape || !rho || !out) return MOE_ERR_NULL;
    if (shape->E_tot < 1 || shape->E_tot > 1024 || shape->T < 0 || shape->k_tot < 1 || occ->tile_m < 1)
        return MOE_ERR_SHAPE;
    int32_t counts[1024];
    const int64_t R = (int64_t)shape->T * shape->k_tot;
    const int64_t per_expert = (R + shape->E_tot - 1) / shape->E_tot;
    const int64_t tiles = (per_expert + occ->tile_m - 1) / occ->tile_m;
    if (tiles > INT32_MAX) return MOE_ERR_SHAPE;
    for (int32_t e = 0; e < shape->E_tot; ++e) counts[e] = (int32_t)tiles;
    return plan_partition(counts, shape->E_tot, occ, limits, shape, rho, out);
}

