// Up-stream stage of the post-router MoE layer on one GPU (Section II-A, steps 1 and 2): the rows of the
// hidden states are collected in routed order (the paper's AllGather; here all tokens are local, so it
// is a gather by the routing permutation), grouped GEMM1 computes the gate and the up projection of
// every routed row with its expert's weights, and the gated activation silu(gate) * up forms x_routed,
// the input of GEMM2 + GatherRS.  The paper leaves this stage unchanged and does not name the
// activation; SiLU gating is the reading taken.
//
// Two launches: gather_rows (one warp per routed row, 16-byte copies), then one persistent kernel,
// one 512-thread CTA per SM, tile = 128 routed rows x 128 intermediate columns:
//   warps 0, 2  TMA producers (one thread each): warp 0 the gathered rows (128 x 64 k), warp 2 the
//               expert's 128 gate rows and 128 up rows of W1 for the same columns (two boxes that form
//               one 256-row B operand), into four 48 KB stages, 128B swizzle;
//   warp 1      issues tcgen05.mma (converged warp, elected lane; M = 128, N = 256, K = 16, bf16 -> fp32): accumulator
//               columns 0..127 are the gate projection, 128..255 the up projection of the same outputs;
//               two accumulator buffers in TMEM;
//   warps 4-15  epilogue: tcgen05.ld of 32 gate and the matching 32 up columns, silu(g) * u in fp32,
//               bf16, two 32-byte stores per row (x_routed rows are contiguous: no scatter here).
// The n-tile index runs fastest in the tile sequence, so the CTAs of a wave share the gathered rows.
// Every wait is bounded like in the fused kernel (status word, no trap).

#include <cuda_bf16.h>

#include <cstring>

#include "moe_internal.h"
#include "sm100_device.cuh"

namespace moe {
namespace {

constexpr int kG1TileN = 128;                                   // intermediate columns per tile
constexpr int kG1ABytes = kMmaM * kBlockK * 2;                  // 16 KB
constexpr int kG1BBytes = 2 * kG1TileN * kBlockK * 2;           // 32 KB: gate rows, then up rows
constexpr int kG1StageBytes = kG1ABytes + kG1BBytes;            // 48 KB
constexpr int kG1Stages = kStageBytesTotal / kG1StageBytes;     // 4
constexpr int kG1EpiWarps = 12;
constexpr int kG1TmemCols = 512;                                // two 256-column accumulators

struct alignas(64) G1Params {
    CUtensorMap tmA;   // h_routed [R, H]            box 64 x 128 rows
    CUtensorMap tmB;   // W1 as [E_tot * 2, I, H]    box 64 x 128 rows x 1 plane
    const int32_t *mtile_expert;
    const int32_t *mtile_first_row;
    const int32_t *mtile_valid;
    const int32_t *S_dev;          // != nullptr: the m-tile count is read here
    __nv_bfloat16 *x_routed;       // [R, I]
    uint32_t *status;
    unsigned long long wait_ns;
    int32_t S;                     // m-tiles of the routing workspace (or their bound with S_dev)
    int32_t sub;                   // 128-row pieces per m-tile (1, or 2 for 256-row m-tiles)
    int32_t sub_rows;              // rows of a piece that may be stored: min(tile_m, 128)
    int32_t I, NT;                 // intermediate size, n-tiles = ceil(I / 128)
    int32_t num_kb, last_ksteps;
};

struct G1Control {
    unsigned long long full[kG1Stages];
    unsigned long long empty[kG1Stages];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    uint32_t tmem_base;
    volatile uint32_t abort;
};

__device__ __forceinline__ bool g1_wait(uint32_t bar, uint32_t parity, G1Control *ctl, unsigned long long deadline,
                                        uint32_t *status, uint32_t detail, uint32_t where)
{
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 63u) == 0u) {
            if (ctl->abort) return false;
            if (globaltimer_ns() > deadline) {
                ctl->abort = 1u;
                report(status, MOE_DEV_TIMEOUT, detail, where);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool g1_wait_warp(uint32_t bar, uint32_t parity, G1Control *ctl, unsigned long long deadline,
                                             uint32_t *status, uint32_t detail, uint32_t where)
{
    uint32_t ok = 1u;
    if ((threadIdx.x & 31u) == 0u) ok = g1_wait(bar, parity, ctl, deadline, status, detail, where) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, ok, 0) != 0u;
}

struct G1Tile {
    int e, row0, valid, n0;
};
// tile g of the sequence: (m-tile, 128-row piece) outer, n-tile inner
__device__ __forceinline__ G1Tile g1_decode(int g, const G1Params &P)
{
    const int piece = g / P.NT;
    const int i_n = g - piece * P.NT;
    const int mu = piece / P.sub;
    const int half = piece - mu * P.sub;
    G1Tile t;
    t.e = __ldg(&P.mtile_expert[mu]);
    t.row0 = __ldg(&P.mtile_first_row[mu]) + half * kMmaM;
    t.valid = max(0, min(P.sub_rows, __ldg(&P.mtile_valid[mu]) - half * kMmaM));
    t.n0 = i_n * kG1TileN;
    return t;
}

// --------------------------------------------------------------------------- gather

// h_routed[r][:] = hidden[perm[r] / k_tot][:], one warp per routed row
__global__ void __launch_bounds__(256)
gather_rows(const uint4 *__restrict__ hidden, const int32_t *__restrict__ perm, int R, int k_tot, int row_vec,
            uint4 *__restrict__ h_routed)
{
    const int r = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5);
    if (r >= R) return;
    const int lane = threadIdx.x & 31;
    const int t = __ldg(&perm[r]) / k_tot;
    const uint4 *src = hidden + (size_t)t * row_vec;
    uint4 *dst = h_routed + (size_t)r * row_vec;
    for (int c = lane; c < row_vec; c += 32) dst[c] = __ldg(&src[c]);
}

// --------------------------------------------------------------------------- GEMM1 + activation

__global__ void __launch_bounds__(kThreads, 1)
moe_gemm1_act_kernel(const __grid_constant__ G1Params P)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    G1Control *ctl = reinterpret_cast<G1Control *>(ring + kStageBytesTotal);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = P.S_dev ? min(__ldg(P.S_dev), P.S) : P.S;
    const int total_tiles = S * P.sub * P.NT;
    const int b = (int)blockIdx.x, stride = (int)gridDim.x;
    const unsigned long long deadline = globaltimer_ns() + P.wait_ns;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kG1Stages; ++i) {
            mbar_init(smem_u32(&ctl->full[i]), 1);
            mbar_init(smem_u32(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[i]), kG1EpiWarps);
        }
        ctl->abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&ctl->tmem_base), kG1TmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0 || warp == 2) {
        // ---------------- TMA producers
        const bool load_a = (warp == 0);
        if (lane == 0 && b < total_tiles) {
            int stage = 0;
            uint32_t phase = 0, armed = 0;
            bool ok = true;
            G1Tile t = g1_decode(b, P);
            for (int g = b; g < total_tiles && ok; g += stride) {
                const G1Tile t_next = g1_decode(min(g + stride, total_tiles - 1), P);   // fetched one tile ahead
                int kx = 0;
                for (int kb = 0; kb < P.num_kb; ++kb, kx += kBlockK) {
                    ok = g1_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, deadline, P.status, (uint32_t)g, 50u);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&ctl->full[stage]);
                    const uint32_t a_dst = smem_u32(ring + stage * kG1StageBytes);
                    if (load_a) {
                        mbar_arrive_expect_tx(full, (uint32_t)kG1StageBytes);
                        tma_load_2d(a_dst, &P.tmA, full, kx, t.row0);
                    } else {
                        tma_load_3d(a_dst + kG1ABytes, &P.tmB, full, kx, t.n0, 2 * t.e);                     // gate rows
                        tma_load_3d(a_dst + kG1ABytes + kG1BBytes / 2, &P.tmB, full, kx, t.n0, 2 * t.e + 1); // up rows
                    }
                    armed |= 1u << stage;
                    if (++stage == kG1Stages) { stage = 0; phase ^= 1u; }
                }
                t = t_next;
            }
            if (!ok) {
                // wind-down: let the copies already issued land before shared memory is released
                const unsigned long long drain = globaltimer_ns() + 2000000ull;
                for (int sidx = 0; sidx < kG1Stages; ++sidx) {
                    if (!(armed & (1u << sidx))) continue;
                    const uint32_t par = (sidx < stage) ? phase : (phase ^ 1u);
                    while (!mbar_try_wait(smem_u32(&ctl->full[sidx]), par) && globaltimer_ns() < drain) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer: the whole warp runs the loop, converged, and one elected lane issues.
        // tcgen05.mma takes its descriptors and addresses from uniform registers, and the tensor pipe buffers
        // little ahead of the MMA it executes: warp-uniform values in warp-uniform control flow spare a move per
        // operand and MMA, a whole k-block (four MMAs and the commit) is one statement with 32-bit descriptor
        // arithmetic, addresses advance by additions, the barrier's first look is the non-suspending test.
        {
            constexpr uint32_t idesc = make_idesc(kMmaM, 2 * kG1TileN);
            constexpr uint32_t kLoStage = (uint32_t)(kG1StageBytes >> 4), kLoB = (uint32_t)(kG1ABytes >> 4);
            const uint32_t lo0 = smem_desc_lo(smem_u32(ring));
            const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
            uint32_t a_lo = lo0, full_bar = full0, empty_bar = empty0;
            int stage = 0, it = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int g = b; g < total_tiles && ok; g += stride, ++it) {
                const int a = it & 1;
                const uint32_t acc_parity = ((uint32_t)(it >> 1) & 1u) ^ 1u;
                if (!__all_sync(0xffffffffu, mbar_test_wait(smem_u32(&ctl->tmem_empty[a]), acc_parity))) {
                    // (every lane polls; the vote keeps `ok`, and with it the loop, provably warp-uniform)
                    ok = __all_sync(0xffffffffu, g1_wait(smem_u32(&ctl->tmem_empty[a]), acc_parity, ctl, deadline, P.status, (uint32_t)g, 51u));
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * 2 * kG1TileN);
                for (int kb = 0; kb < P.num_kb; ++kb) {
                    if (!__all_sync(0xffffffffu, mbar_test_wait(full_bar, phase))) {
                        ok = __all_sync(0xffffffffu, g1_wait(full_bar, phase, ctl, deadline, P.status, (uint32_t)g, 52u));
                        if (!ok) break;
                    }
                    tc_fence_after();
                    if (elect_one_sync()) {
                        if (kb < P.num_kb - 1 || P.last_ksteps == kBlockK / kUmmaK) {
                            tc_kblock_bf16(d_tmem, a_lo, a_lo + kLoB, idesc, kb > 0 ? 1u : 0u, empty_bar);
                        } else {
                            const uint64_t a_desc = ((uint64_t)kSmemDescHi << 32) | a_lo, b_desc = a_desc + kLoB;
                            for (int k = 0; k < P.last_ksteps; ++k)
                                tc_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                            (k > 0 || kb > 0) ? 1u : 0u);
                            tc_commit(empty_bar);
                        }
                    }
                    a_lo += kLoStage;
                    full_bar += 8u;
                    empty_bar += 8u;
                    if (++stage == kG1Stages) {
                        stage = 0;
                        phase ^= 1u;
                        a_lo = lo0;
                        full_bar = full0;
                        empty_bar = empty0;
                    }
                }
                __syncwarp();
                if (ok && elect_one_sync()) tc_commit(smem_u32(&ctl->tmem_full[a]));
            }
        }
        __syncwarp();
    } else if (warp >= 4 && warp < 4 + kG1EpiWarps) {
        // ---------------- epilogue: four 32-column rounds per tile, dealt 2 / 1 / 1 to the column groups
        const int q4 = warp & 3;
        const int grp = (warp - 4) >> 2;
        const int round0 = grp == 0 ? 0 : grp + 1;
        const int n_rounds = grp == 0 ? 2 : 1;
        const int row_in_tile = q4 * 32 + lane;
        int it = 0;
        for (int g = b; g < total_tiles; g += stride, ++it) {
            const G1Tile t = g1_decode(g, P);
            const int a = it & 1;
            const bool ok = g1_wait_warp(smem_u32(&ctl->tmem_full[a]), (uint32_t)(it >> 1) & 1u, ctl, deadline, P.status,
                                         (uint32_t)g, 53u);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(a * 2 * kG1TileN);
            const bool row_ok = row_in_tile < t.valid;
            __nv_bfloat16 *dst_row = P.x_routed + (size_t)(t.row0 + row_in_tile) * (size_t)P.I + t.n0;
#pragma unroll 1
            for (int rr = 0; rr < n_rounds; ++rr) {
                const int col = (round0 + rr) * 32;
                uint32_t gt[32], up[32];
                tmem_ld_32x32(taddr + (uint32_t)col, gt);
                tmem_ld_32x32(taddr + (uint32_t)(kG1TileN + col), up);
                tmem_ld_wait(gt);
                tmem_ld_wait(up);
                if (rr == n_rounds - 1) {
                    // everything this warp needs of the accumulator is in registers: hand the buffer back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[a]));
                }
                if (row_ok) {
#pragma unroll
                    for (int v = 0; v < 2; ++v) {
                        if (t.n0 + col + v * 16 < P.I) {
                            uint32_t w[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float g0 = __uint_as_float(gt[v * 16 + 2 * i]), g1 = __uint_as_float(gt[v * 16 + 2 * i + 1]);
                                const float u0 = __uint_as_float(up[v * 16 + 2 * i]), u1 = __uint_as_float(up[v * 16 + 2 * i + 1]);
                                // silu(z) * u = z / (1 + exp(-z)) * u
                                const float x0 = g0 / (1.0f + __expf(-g0)) * u0;
                                const float x1 = g1 / (1.0f + __expf(-g1)) * u1;
                                __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
                                w[i] = *reinterpret_cast<uint32_t *>(&h);
                            }
                            st_global_v8(dst_row + col + v * 16, w);
                        }
                    }
                }
            }
        }
    }
    // ---------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kG1TmemCols);
    }
}

size_t g1_smem_bytes() { return (size_t)kStageBytesTotal + 1024 + ((sizeof(G1Control) + 127) & ~(size_t)127); }

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace
}  // namespace moe

using namespace moe;

extern "C" int32_t moe_gemm1_workspace_bytes(const moe_shape *s, size_t *h_routed_bytes)
{
    if (!s || !h_routed_bytes) return MOE_ERR_NULL;
    if (s->T < 0 || s->k_tot < 1 || s->H < 1) return MOE_ERR_SHAPE;
    *h_routed_bytes = (((size_t)s->T * s->k_tot * s->H * 2) + 15) / 16 * 16 + 16;
    return MOE_OK;
}

extern "C" int32_t moe_gemm1_act(moe_handle *h, const void *hidden, const void *W1, const moe_shape *s,
                                 int32_t tile_m, const moe_routing *r, int32_t n_mtiles, void *h_routed_ws,
                                 void *x_routed, uint32_t *status_dev, void *stream)
{
    if (!h || !s || !r || !status_dev) return MOE_ERR_NULL;
    if (s->T < 0 || s->H < 64 || s->H % 16 != 0 || s->I < 16 || s->I % 16 != 0 || s->E_tot < 1 || s->k_tot < 1 ||
        (int64_t)s->T * s->k_tot >= (int64_t)1 << 30)
        return MOE_ERR_SHAPE;
    if (tile_m != 64 && tile_m != 128 && tile_m != 256) return MOE_ERR_UNSUPPORTED;
    if (s->T == 0) return MOE_OK;
    if (!hidden || !W1 || !h_routed_ws || !x_routed) return MOE_ERR_NULL;
    if (!aligned(hidden, 16) || !aligned(W1, 16) || !aligned(h_routed_ws, 16) || !aligned(x_routed, 32) ||
        !aligned(status_dev, 16))
        return MOE_ERR_ALIGN;
    const bool counts_on_device = (n_mtiles == MOE_MTILES_ON_DEVICE);
    if (counts_on_device) n_mtiles = r->max_mtiles;
    if (n_mtiles < 0 || n_mtiles > r->max_mtiles) return MOE_ERR_SHAPE;
    if (const int32_t rc = moe::require_handle_device(h, "moe_gemm1_act")) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int R = s->T * s->k_tot;

    G1Params p;
    memset(&p, 0, sizeof p);
    p.mtile_expert = r->mtile_expert;
    p.mtile_first_row = r->mtile_first_row;
    p.mtile_valid = r->mtile_valid;
    p.S_dev = counts_on_device ? r->tiles + s->E_tot : nullptr;
    p.x_routed = static_cast<__nv_bfloat16 *>(x_routed);
    p.status = status_dev;
    p.wait_ns = h->wait_ns;
    p.S = n_mtiles;
    p.sub = tile_m == 256 ? 2 : 1;
    p.sub_rows = tile_m < kMmaM ? tile_m : kMmaM;
    p.I = s->I;
    p.NT = (s->I + kG1TileN - 1) / kG1TileN;
    p.num_kb = (s->H + kBlockK - 1) / kBlockK;
    p.last_ksteps = (s->H - (p.num_kb - 1) * kBlockK) / kUmmaK;
    if ((int64_t)n_mtiles * p.sub * p.NT >= (int64_t)1 << 31) return MOE_ERR_SHAPE;

    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(h->encode_tiled);
    {
        cuuint64_t dims[2] = {(cuuint64_t)s->H, (cuuint64_t)R};
        cuuint64_t strides[1] = {(cuuint64_t)s->H * 2};
        cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)kMmaM};
        cuuint32_t es[2] = {1, 1};
        CUresult cr = encode(&p.tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, h_routed_ws, dims, strides, box, es,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) {
            snprintf(h->err, sizeof h->err, "cuTensorMapEncodeTiled(h_routed) failed: %d", (int)cr);
            return MOE_ERR_CUDA;
        }
    }
    {
        // W1 [E_tot][2][I][H] seen as [E_tot * 2 planes][I rows][H]: rows past I of a plane read zeros
        cuuint64_t dims[3] = {(cuuint64_t)s->H, (cuuint64_t)s->I, (cuuint64_t)s->E_tot * 2};
        cuuint64_t strides[2] = {(cuuint64_t)s->H * 2, (cuuint64_t)s->H * 2 * (cuuint64_t)s->I};
        cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)kG1TileN, 1};
        cuuint32_t es[3] = {1, 1, 1};
        CUresult cr = encode(&p.tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(W1), dims, strides, box, es,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) {
            snprintf(h->err, sizeof h->err, "cuTensorMapEncodeTiled(W1) failed: %d", (int)cr);
            return MOE_ERR_CUDA;
        }
    }

    // gather (the rows of a token are read k_tot times, from L2 after the first)
    const int row_vec = s->H * 2 / 16;
    const unsigned gather_blocks = (unsigned)(((int64_t)R * 32 + 255) / 256);
    gather_rows<<<gather_blocks, 256, 0, st>>>(static_cast<const uint4 *>(hidden), r->perm, R, s->k_tot, row_vec,
                                               static_cast<uint4 *>(h_routed_ws));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e, "gather_rows launch");

    const size_t smem = g1_smem_bytes();
    e = cudaFuncSetAttribute(moe_gemm1_act_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(h, e, "gemm1 shared memory attribute");
    const int64_t tiles_bound = (int64_t)n_mtiles * p.sub * p.NT;
    const int grid = (int)(tiles_bound < h->G ? (tiles_bound > 0 ? tiles_bound : 1) : h->G);
    moe_gemm1_act_kernel<<<grid, kThreads, smem, st>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e, "gemm1 launch");
    return MOE_OK;
}
