/*
 * GEMM1 + gated activation reference (CPU oracle, test infrastructure).
 *
 * Only the tests and the benchmark's CPU legs may build or call this file.  It shares no code with
 * the CUDA path.
 *
 * What it computes (paper Section II-A, steps 1 and 2 of the post-router MoE layer: "grouped GEMM1
 * performs the gate and up projections", then "a gated activation combines the two projections to
 * form the intermediate representation for each expert"), for the routed row r that belongs to
 * assignment f = perm[r] (token t = f div k_tot, expert e = topk_idx[f]):
 *
 *     g[i] = sum_h hidden[t][h] * W1[e][0][i][h]          (gate projection)
 *     u[i] = sum_h hidden[t][h] * W1[e][1][i][h]          (up projection)
 *     x_routed[r][i] = silu(g[i]) * u[i],   silu(z) = z / (1 + exp(-z))
 *
 * The paper does not name the activation; SiLU gating (SwiGLU) is the reading taken, the one the
 * three model families of its evaluation use.  The collection of the participating input rows
 * (AllGather in the paper) is the indexing hidden[t] above: on one GPU all tokens are local.
 * Plain loops in that order: per row, per intermediate column i, two sequential dot products over
 * h in fp32 (the _f64 variant carries dot products and activation in double).  Inputs are bf16 bit
 * patterns; the result is returned unrounded.  OpenMP only spreads rows over cores.
 */

#include <math.h>
#include <stdint.h>
#include <string.h>

static float g1_bf16_to_f32(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/*
 * rows : list of n_rows routed-row ids to evaluate (NULL = rows 0..n_rows-1).
 * W1   : [E_tot][2][I][H], plane 0 = gate, plane 1 = up, the contraction index h contiguous.
 * out  : [n_rows][I] fp32.
 * Returns 0, or -1 when an index is out of range (nothing is written for that row).
 */
int moe_ref_gemm1_act_f32(const uint16_t *hidden, const uint16_t *W1, const int32_t *topk_idx,
                          const int32_t *perm, int T, int H, int I, int E_tot, int k_tot,
                          const int32_t *rows, int n_rows, float *out)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int q = 0; q < n_rows; ++q) {
        int r = rows ? rows[q] : q;
        if (r < 0 || r >= T * k_tot) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        int f = perm[r];
        int e = (f >= 0 && f < T * k_tot) ? topk_idx[f] : -1;
        if (e < 0 || e >= E_tot) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        int t = f / k_tot;
        const uint16_t *hrow = hidden + (size_t)t * H;
        const uint16_t *Wg = W1 + ((size_t)e * 2 + 0) * I * H;
        const uint16_t *Wu = W1 + ((size_t)e * 2 + 1) * I * H;
        for (int i = 0; i < I; ++i) {
            float g = 0.0f, u = 0.0f;
            for (int h = 0; h < H; ++h) g = g + g1_bf16_to_f32(hrow[h]) * g1_bf16_to_f32(Wg[(size_t)i * H + h]);
            for (int h = 0; h < H; ++h) u = u + g1_bf16_to_f32(hrow[h]) * g1_bf16_to_f32(Wu[(size_t)i * H + h]);
            float s = g / (1.0f + expf(-g));
            out[(size_t)q * I + i] = s * u;
        }
    }
    return bad ? -1 : 0;
}

/* Same loops in double; out is [n_rows][I] double. */
int moe_ref_gemm1_act_f64(const uint16_t *hidden, const uint16_t *W1, const int32_t *topk_idx,
                          const int32_t *perm, int T, int H, int I, int E_tot, int k_tot,
                          const int32_t *rows, int n_rows, double *out)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int q = 0; q < n_rows; ++q) {
        int r = rows ? rows[q] : q;
        if (r < 0 || r >= T * k_tot) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        int f = perm[r];
        int e = (f >= 0 && f < T * k_tot) ? topk_idx[f] : -1;
        if (e < 0 || e >= E_tot) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        int t = f / k_tot;
        const uint16_t *hrow = hidden + (size_t)t * H;
        const uint16_t *Wg = W1 + ((size_t)e * 2 + 0) * I * H;
        const uint16_t *Wu = W1 + ((size_t)e * 2 + 1) * I * H;
        for (int i = 0; i < I; ++i) {
            double g = 0.0, u = 0.0;
            for (int h = 0; h < H; ++h) g = g + (double)g1_bf16_to_f32(hrow[h]) * (double)g1_bf16_to_f32(Wg[(size_t)i * H + h]);
            for (int h = 0; h < H; ++h) u = u + (double)g1_bf16_to_f32(hrow[h]) * (double)g1_bf16_to_f32(Wu[(size_t)i * H + h]);
            double s = g / (1.0 + exp(-g));
            out[(size_t)q * I + i] = s * u;
        }
    }
    return bad ? -1 : 0;
}
