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

// ---- co-resident family with a bandwidth-coupled service rate (this library's re-derivation; Section III-E
// asks a new kernel family for its own o_comm, legal range and service rate).  Capacity is counted in warps:
// a communication tile is `warps_cta` quanta; N warps streaming together take rho * max(N, n_sat) / n_sat per
// quantum; a co-resident warp counts as 1/gamma dedicated warps while the GEMM runs and stretches the compute
// wave by beta (and by `order` when the tile sequence has to be split-major for it).

struct CoModel {
    int64_t warps_cta, n_sat;        // n_sat = INT64_MAX: never saturated
    int64_t quanta_tile;             // pieces a communication tile is handed out in (>= 1)
    int64_t beta_q, gamma_q, order_q;
};

inline int64_t coupled_rho(int64_t rho_q, int64_t n, int64_t n_sat)
{
    if (n <= n_sat) return rho_q;
    const unsigned __int128 num = (unsigned __int128)rho_q * (unsigned __int128)n;
    return (int64_t)((num + (unsigned __int128)(n_sat - 1)) / (unsigned __int128)n_sat);
}

// full waves of n_workers, then a partial wave: each takes rho(streams in that wave)
inline int64_t coupled_service(int64_t rho_q, int64_t quanta, int64_t n_workers, int64_t n_sat)
{
    const int64_t full = quanta / n_workers, rest = quanta - full * n_workers;
    return full * coupled_rho(rho_q, n_workers, n_sat) + (rest ? coupled_rho(rho_q, rest, n_sat) : 0);
}

inline bool evaluate_co(int32_t C, int32_t w, int64_t Wc, int64_t Wm, int32_t L, int32_t G, int32_t o_comp,
                        int32_t o_comm, int32_t slot_sms, int64_t rho_q, const CoModel &m, Candidate *out)
{
    const int32_t R = (C + o_comm - 1) / o_comm;
    const int64_t P = G > R ? (int64_t)o_comp * ((G - R) / slot_sms) : 0;
    if (P <= 0) return false;
    const int64_t n_sm = P * slot_sms / o_comp;
    const int64_t tau_q = ((int64_t)1 << kRhoShift) + w * m.beta_q + ((w > 0 && L > 1) ? m.order_q : 0);
    const int64_t Wq = Wm * m.quanta_tile;
    const int64_t n_early = (int64_t)C * m.warps_cta + w * n_sm;
    const int64_t n_eff = (int64_t)C * m.warps_cta + ((w * n_sm) << kRhoShift) / m.gamma_q;
    const int64_t A_last = ceil_div64((int64_t)L * Wc, P) * tau_q;
    int64_t backlog;
    if (n_eff <= 0) {
        backlog = (int64_t)(L - 1) * Wq;
    } else {
        const int64_t q_wave = coupled_rho(rho_q, n_early, m.n_sat);
        const int64_t q = q_wave * ceil_div64(Wq, n_eff);
        int64_t F = 0;
        for (int32_t s = 0; s + 1 < L; ++s) {
            // without co-resident warps the tiles run m-tile-major: no split is published before the last
            const int64_t A = w > 0 ? ceil_div64((int64_t)(s + 1) * Wc, P) * tau_q : A_last;
            F = (A > F ? A : F) + q;
        }
        backlog = 0;
        if (F > A_last && q_wave > 0) {
            backlog = ceil_div64(F - A_last, q_wave) * n_eff;
            if (backlog > (int64_t)(L - 1) * Wq) backlog = (int64_t)(L - 1) * Wq;
        }
    }
    const int64_t n_tail = ((int64_t)C + n_sm) * m.warps_cta + w * n_sm;
    out->T_q = A_last + coupled_service(rho_q, backlog + Wq, n_tail, m.n_sat);
    out->delta = ceil_div64(Wc, P) * P - Wc;
    out->C = C;
    out->R = R;
    out->P = (int32_t)P;
    return true;
}

// ---- tile-level readiness for the static partition: Eq. 9 applied to every communication tile.
// idx[ct] = compute tile of the split whose completion makes communication tile ct (static map order,
// token-tiles rank-major, column tile fastest) ready; the rows of the last non-empty expert gate the tokens
// in order.  Returns the number of communication tiles written, or -1 when `cap` is too small.
inline int32_t comm_tile_ready_index(const int32_t *tiles, int32_t n_experts, int64_t g, int64_t M, int32_t D,
                                     int64_t split_w, int64_t T_N, int64_t T_Mc, int64_t T_Nc, int32_t *idx, int32_t cap)
{
    int64_t S = 0, n_last = 0;
    for (int32_t e = 0; e < n_experts; ++e) {
        S += tiles[e];
        if (tiles[e] > 0) n_last = tiles[e];
    }
    const int64_t NT = ceil_div64(split_w, T_N), n_col = ceil_div64(split_w, T_Nc);
    const int64_t blk = ceil_div64(M, D);
    int32_t n = 0;
    for (int32_t d = 0; d < D; ++d) {
        int64_t own = M - (int64_t)d * blk;
        if (own > blk) own = blk;
        if (own <= 0) continue;
        for (int64_t ti = 0; ti < ceil_div64(own, T_Mc); ++ti) {
            const int64_t t_hi = (int64_t)d * blk + ((ti + 1) * T_Mc < own ? (ti + 1) * T_Mc : own);
            int64_t i_j = M > 0 ? ceil_div64(n_last * t_hi, M) - 1 : 0;
            if (i_j < 0) i_j = 0;
            const int64_t mu = S - n_last + i_j;
            for (int64_t c = 0; c < n_col; ++c) {
                const int64_t hi_col = (c + 1) * T_Nc < split_w ? (c + 1) * T_Nc : split_w;
                const int64_t n_hi = ceil_div64(hi_col, T_N) - 1;
                if (n >= cap) return -1;
                idx[n++] = (int32_t)((mu * g + (g - 1)) * NT + n_hi);
            }
        }
    }
    return n;
}

// F_{s,v} = max(max_{ct < min(vC+C, W_comm)} a_{s,ct}, F_{s,v-1}) + rho, a_{s,ct} = floor((s W_comp + idx) / P) + 1.
// `pmax[ct]` = max(idx[0..ct]).  Once the served front F has passed the readiness of the split's very last
// tile, every remaining wave of the split just adds rho.
inline bool evaluate_tile_level(int32_t C, const int32_t *pmax, int32_t Wm, int64_t Wc, int32_t L, int32_t G,
                                int32_t o_comp, int32_t o_comm, int32_t slot_sms, int64_t rho_q, Candidate *out)
{
    const int32_t R = (C + o_comm - 1) / o_comm;
    const int64_t P = G > R ? (int64_t)o_comp * ((G - R) / slot_sms) : 0;
    if (P <= 0) return false;
    int64_t F = 0;
    const int32_t waves = (Wm + C - 1) / C;
    for (int32_t s = 0; s < L && Wm > 0; ++s) {
        const int64_t a_end = (((int64_t)s * Wc + pmax[Wm - 1]) / P + 1) << kRhoShift;   // the split's last tile ready
        int64_t q = ((int64_t)s * Wc + pmax[0]) / P;       // floor((s W_comp + top) / P), carried: top only grows
        for (int32_t v = 0; v < waves; ++v) {
            if (F >= a_end) {                               // nothing of this split is waited for any more
                F += (int64_t)(waves - v) * rho_q;
                break;
            }
            const int32_t last = (v + 1) * C < Wm ? (v + 1) * C - 1 : Wm - 1;
            const int64_t num = (int64_t)s * Wc + pmax[last];
            while ((q + 1) * P <= num) ++q;
            const int64_t a = (q + 1) << kRhoShift;
            F = (a > F ? a : F) + rho_q;
        }
    }
    out->T_q = F;
    out->delta = ceil_div64(Wc, P) * P - Wc;
    out->C = C;
    out->R = R;
    out->P = (int32_t)P;
    return true;
}

inline int64_t quantise(double v) { return (int64_t)(v * (double)(1 << kRhoShift) + 0.5); }

constexpr int32_t kMaxCommTilesTileLevel = 4096;   // communication tiles per split the tile-level model handles

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
    int32_t best_w = 0;
    const bool co_family = dh && rho->comm_warps_per_cta > 0;
    const bool tile_level = !dh && limits->dep_model == MOE_DEP_TILE;
    if (co_family) {
        // product set (C, w): w = 0 with every legal C, w >= 1 with C up to C_co_max; lexicographic minimum of
        // (T, Delta_comp, w, C) -- ascending w then C, so only a strict improvement of (T, Delta) replaces
        if (!(rho->co_gamma >= 1.0) || rho->co_gamma > 1.0e3 || !(rho->co_beta >= 0.0) || rho->co_beta > 1.0e3 ||
            !(rho->co_order >= 0.0) || rho->co_order > 1.0e3 || rho->n_sat_warps < 0 || rho->comm_quanta_per_tile < 0)
            return MOE_ERR_SHAPE;
        CoModel m;
        m.warps_cta = rho->comm_warps_per_cta;
        m.quanta_tile = rho->comm_quanta_per_tile > 0 ? rho->comm_quanta_per_tile : rho->comm_warps_per_cta;
        // one warp serves one piece of a tile in rho * warps_cta / quanta_tile (a dedicated CTA a tile in rho);
        // from here on rho_q is that per-piece time (the plan still reports the per-tile rho)
        const int64_t rho_tile_q = rho_q;
        const int64_t rho_q = (int64_t)(((unsigned __int128)rho_tile_q * (unsigned __int128)m.warps_cta) / (unsigned __int128)m.quanta_tile);
        m.n_sat = rho->n_sat_warps > 0 ? rho->n_sat_warps : INT64_MAX;
        m.beta_q = quantise(rho->co_beta);
        m.gamma_q = quantise(rho->co_gamma);
        m.order_q = quantise(rho->co_order);
        const bool forced_C = limits->force_comm_ctas > 0 || limits->selector_off;
        const int32_t C_forced = limits->force_comm_ctas > 0 ? limits->force_comm_ctas : limits->default_C;
        if (forced_C && C_forced < 1) return MOE_ERR_PLAN_INFEASIBLE;
        const int32_t w_top = limits->co_warps_max > 0 ? limits->co_warps_max : 0;
        const int32_t w_lo = limits->force_co_warps >= 0 ? (limits->force_co_warps < w_top ? limits->force_co_warps : w_top) : 0;
        const int32_t w_hi = limits->force_co_warps >= 0 ? w_lo : w_top;
        // The same integers as evaluate_co(), cheaper: ceilings that only move one way as C grows are carried
        // and corrected with multiply-compare steps, quotients by n_sat / gamma / rho come from a double estimate
        // made exact, and a candidate whose compute phase alone (A_{L-1}, which only grows with C) plus the least
        // any tail can take already exceeds the incumbent ends the scan of its w.
        const int64_t Wq = Wm * m.quanta_tile;
        const int64_t n_max = (int64_t)G * slot * (m.warps_cta + w_top) + (int64_t)limits->C_max * m.warps_cta;
        const bool fast = !forced_C && rho_q > 0 && rho_q < ((int64_t)1 << 40) && n_max < ((int64_t)1 << 20) &&
                          (int64_t)L * Wc < ((int64_t)1 << 40) && Wq < ((int64_t)1 << 40) && m.gamma_q < ((int64_t)1 << 31) &&
                          m.beta_q < ((int64_t)1 << 31) && m.order_q < ((int64_t)1 << 31);
        const double inv_nsat = 1.0 / (double)m.n_sat, inv_gamma = 1.0 / (double)m.gamma_q, inv_rho = rho_q > 0 ? 1.0 / (double)rho_q : 0.0;
        auto rho_of = [&](int64_t n) -> int64_t {          // coupled_rho with 64-bit products (fast path only)
            if (n <= m.n_sat) return rho_q;
            const int64_t num = rho_q * n;
            int64_t q = (int64_t)((double)num * inv_nsat);
            while (q * m.n_sat < num) ++q;
            while (q > 0 && (q - 1) * m.n_sat >= num) --q;
            return q;
        };
        // least time any tail needs: the last split's quanta at the bandwidth, and one wave
        int64_t lb_tail = Wq > 0 ? rho_q : 0;
        if (fast && m.n_sat != INT64_MAX) {
            const int64_t bw = (int64_t)(((unsigned __int128)rho_q * (unsigned __int128)Wq) / (unsigned __int128)m.n_sat);
            if (bw > lb_tail) lb_tail = bw;
        }
        for (int32_t w = w_lo; w <= w_hi; ++w) {
            int32_t C_lo = 1, C_hi = limits->C_max;
            if (w > 0 && limits->C_co_max < C_hi) C_hi = limits->C_co_max;
            if (forced_C) C_lo = C_hi = C_forced;
            if (!fast) {
                for (int32_t C = C_lo; C <= C_hi; ++C) {
                    Candidate c;
                    if (!evaluate_co(C, w, Wc, Wm, L, G, o_comp, o_comm, slot, rho_q, m, &c)) break;   // P only falls
                    // lower end of the legal set: co-resident warps need a compute phase of co_min_waves waves
                    if (w > 0 && limits->force_co_warps < 0 && ceil_div64((int64_t)L * Wc, c.P) < limits->co_min_waves) continue;
                    if (!have || c.T_q < best.T_q || (c.T_q == best.T_q && c.delta < best.delta)) {
                        best = c;
                        best_w = w;
                        have = true;
                    }
                }
                continue;
            }
            const int64_t tau_q = ((int64_t)1 << kRhoShift) + w * m.beta_q + ((w > 0 && L > 1) ? m.order_q : 0);
            int64_t qa[MOE_MAX_L];
            int64_t P_prev = 0, n_sm = 0, co_eff = 0;
            for (int32_t C = C_lo; C <= C_hi; ++C) {
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
                    n_sm = (o_comp == 1) ? P * slot : P * slot / o_comp;
                    // floor(w * n_sm * 2^20 / gamma_q): a co-resident warp counts as 1/gamma dedicated warps
                    const int64_t t = (w * n_sm) << kRhoShift;
                    co_eff = (int64_t)((double)t * inv_gamma);
                    while (co_eff * m.gamma_q > t) --co_eff;
                    while ((co_eff + 1) * m.gamma_q <= t) ++co_eff;
                }
                const int64_t A_last = qa[L - 1] * tau_q;
                if (have && A_last + lb_tail > best.T_q) break;     // A_last only grows with C: nothing further can win
                // lower end of the legal set: co-resident warps need a compute phase of co_min_waves waves
                if (w > 0 && limits->force_co_warps < 0 && qa[L - 1] < limits->co_min_waves) continue;
                const int64_t n_early = (int64_t)C * m.warps_cta + w * n_sm;
                const int64_t n_eff = (int64_t)C * m.warps_cta + co_eff;
                int64_t backlog;
                if (n_eff <= 0) {
                    backlog = (int64_t)(L - 1) * Wq;
                } else {
                    const int64_t q_wave = rho_of(n_early);
                    backlog = 0;
                    if (L > 1) {
                        const int64_t q = q_wave * ceil_div64(Wq, n_eff);
                        int64_t F = 0;
                        for (int32_t s = 0; s + 1 < L; ++s) {
                            const int64_t A = w > 0 ? qa[s] * tau_q : A_last;   // m-tile-major order: nothing is early
                            F = (A > F ? A : F) + q;
                        }
                        if (F > A_last) {
                            const int64_t num = F - A_last;
                            int64_t wv = (int64_t)((double)num * (q_wave == rho_q ? inv_rho : 1.0 / (double)q_wave));
                            while (wv * q_wave < num) ++wv;
                            while (wv > 0 && (wv - 1) * q_wave >= num) --wv;
                            backlog = wv * n_eff;
                            if (backlog > (int64_t)(L - 1) * Wq) backlog = (int64_t)(L - 1) * Wq;
                        }
                    }
                }
                const int64_t n_tail = ((int64_t)C + n_sm) * m.warps_cta + w * n_sm;
                const int64_t X = backlog + Wq;
                int64_t full = 0, rest = X;
                if (X >= 8 * n_tail) {
                    full = X / n_tail;
                    rest = X - full * n_tail;
                } else {
                    while (rest >= n_tail) { rest -= n_tail; ++full; }
                }
                const int64_t T_q = A_last + (full ? full * rho_of(n_tail) : 0) + (rest ? rho_of(rest) : 0);
                const int64_t delta = qa[0] * P - Wc;
                if (!have || T_q < best.T_q || (T_q == best.T_q && delta < best.delta)) {
                    best.T_q = T_q;
                    best.delta = delta;
                    best.C = C;
                    best.R = R;
                    best.P = (int32_t)P;
                    best_w = w;
                    have = true;
                }
            }
        }
    } else if (tile_level) {
        int32_t idx[kMaxCommTilesTileLevel];
        const int32_t n = comm_tile_ready_index(routed_tile_counts, n_experts, shape->TP, shape->T, shape->EP, split_w,
                                                occ->tile_n, occ->comm_tile_m, occ->comm_tile_n, idx, kMaxCommTilesTileLevel);
        if (n < 0 || n != (int32_t)Wm) return MOE_ERR_SHAPE;
        for (int32_t ct = 1; ct < n; ++ct)                 // prefix maximum: readiness of "every tile up to ct"
            if (idx[ct] < idx[ct - 1]) idx[ct] = idx[ct - 1];
        if (limits->force_comm_ctas > 0 || limits->selector_off) {
            const int32_t C = limits->force_comm_ctas > 0 ? limits->force_comm_ctas : limits->default_C;
            if (C < 1) return MOE_ERR_PLAN_INFEASIBLE;
            have = evaluate_tile_level(C, idx, n, Wc, L, G, o_comp, o_comm, slot, rho_q, &best);
        } else {
            for (int32_t C = 1; C <= limits->C_max; ++C) {
                Candidate c;
                if (!evaluate_tile_level(C, idx, n, Wc, L, G, o_comp, o_comm, slot, rho_q, &c)) break;
                if (!have || c.T_q < best.T_q || (c.T_q == best.T_q && c.delta < best.delta)) {
                    best = c;
                    have = true;
                }
            }
        }
    } else if (limits->force_comm_ctas > 0 || limits->selector_off) {
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
    out->co_warps = best_w;
    // without the co-resident model an explicit request is still honoured (the launch validates it)
    if (!co_family && dh && limits->co_warps_max > 0 && limits->force_co_warps > 0)
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

