/*
 * GEMM2 + combine reference (CPU oracle, test infrastructure).
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may build or call
 * this file.  It shares no code with the CUDA path.
 *
 * What it computes (paper Section II-A, step 3 "GEMM2+GatherRS": grouped GEMM2 projects each
 * routed row back to the hidden dimension, GatherRS sums the top-k expert contributions of
 * every token and writes the token's output to the rank that owns it):
 *
 *     out[t][h] = sum_j  w[t][j] * ( sum_i x_routed[inv_perm[t*k_tot + j]][i] * W2[e(t,j)][h][i] )
 *
 * written as the plain loops of that definition: per token, per selected expert in slot
 * order j = 0..k_tot-1, per output column h, a sequential dot product over i.  Inputs are
 * bf16 bit patterns (uint16); every product and sum is fp32 (the _f64 variant carries the
 * dot product and the token sum in double, to bound this file's own rounding).  There is no
 * blocking, no reordering and no vectorisation hint; OpenMP only spreads tokens over cores.
 * Tensor-parallel shards do not appear: the reference sums over the whole of I.
 * The split of tokens over destination ranks (token t belongs to rank t div ceil(T/EP)) is
 * pure indexing and is done by the caller.
 */

#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static float bf16_to_f32(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* round-to-nearest-even fp32 -> bf16 bit pattern (finite inputs) */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

int moe_ref_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Sets the number of threads the loops below may use (for the single-thread timing beside the
 * all-cores one); returns the previous maximum.  No effect without OpenMP. */
int moe_ref_set_threads(int n)
{
#ifdef _OPENMP
    const int before = omp_get_max_threads();
    if (n >= 1) omp_set_num_threads(n);
    return before;
#else
    (void)n;
    return 1;
#endif
}

/*
 * tokens: list of n_tokens token ids to evaluate (NULL = tokens 0..n_tokens-1).
 * out   : [n_tokens][H] fp32, row r belongs to tokens[r].
 * W2    : [E_tot][H][I] (the contraction index i is contiguous).
 * Returns 0, or -1 when an index is out of range (nothing is written for that token).
 */
int moe_ref_gemm2_combine_f32(const uint16_t *x_routed, const uint16_t *W2,
                              const int32_t *topk_idx, const float *topk_w,
                              const int32_t *inv_perm,
                              int T, int H, int I, int E_tot, int k_tot,
                              const int32_t *tokens, int n_tokens, float *out)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_tokens; ++r) {
        int t = tokens ? tokens[r] : r;
        if (t < 0 || t >= T) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        float *acc = out + (size_t)r * H;
        for (int h = 0; h < H; ++h) acc[h] = 0.0f;
        for (int j = 0; j < k_tot; ++j) {
            int e = topk_idx[(size_t)t * k_tot + j];
            int row = inv_perm[(size_t)t * k_tot + j];
            if (e < 0 || e >= E_tot || row < 0 || row >= T * k_tot) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            float w = topk_w[(size_t)t * k_tot + j];
            const uint16_t *x = x_routed + (size_t)row * I;
            const uint16_t *We = W2 + (size_t)e * H * I;
            for (int h = 0; h < H; ++h) {
                const uint16_t *wrow = We + (size_t)h * I;
                float dot = 0.0f;
                for (int i = 0; i < I; ++i)
                    dot = dot + bf16_to_f32(x[i]) * bf16_to_f32(wrow[i]);
                acc[h] = acc[h] + w * dot;
            }
        }
    }
    return bad ? -1 : 0;
}

/* Same loops with double accumulation; out is [n_tokens][H] double. */
int moe_ref_gemm2_combine_f64(const uint16_t *x_routed, const uint16_t *W2,
                              const int32_t *topk_idx, const float *topk_w,
                              const int32_t *inv_perm,
                              int T, int H, int I, int E_tot, int k_tot,
                              const int32_t *tokens, int n_tokens, double *out)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_tokens; ++r) {
        int t = tokens ? tokens[r] : r;
        if (t < 0 || t >= T) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        double *acc = out + (size_t)r * H;
        for (int h = 0; h < H; ++h) acc[h] = 0.0;
        for (int j = 0; j < k_tot; ++j) {
            int e = topk_idx[(size_t)t * k_tot + j];
            int row = inv_perm[(size_t)t * k_tot + j];
            if (e < 0 || e >= E_tot || row < 0 || row >= T * k_tot) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            double w = (double)topk_w[(size_t)t * k_tot + j];
            const uint16_t *x = x_routed + (size_t)row * I;
            const uint16_t *We = W2 + (size_t)e * H * I;
            for (int h = 0; h < H; ++h) {
                const uint16_t *wrow = We + (size_t)h * I;
                double dot = 0.0;
                for (int i = 0; i < I; ++i)
                    dot = dot + (double)bf16_to_f32(x[i]) * (double)bf16_to_f32(wrow[i]);
                acc[h] = acc[h] + w * dot;
            }
        }
    }
    return bad ? -1 : 0;
}

/* Round an fp32 array to bf16 bit patterns, nearest even. */
void moe_ref_round_bf16(const float *in, uint16_t *out, long n)
{
    for (long i = 0; i < n; ++i) out[i] = f32_to_bf16_rne(in[i]);
}
