// Fused grouped GEMM2 + GatherRS combine for sm_100a: one persistent launch, one CTA per SM,
// role by blockIdx.
//
//   blockIdx <  C : communication CTA c (Section II-B: consumes published results; the same
//                   C CTAs serve all splits in sequence; CTA c takes communication tiles
//                   c, c+C, ... of a split -- or, with drain help, its warps pull token ranges
//                   from a queue per split that former compute CTAs also serve).
//   blockIdx >= C : compute CTA b = blockIdx - C (Section III-C: takes global tiles
//                   b, b+P, b+2P, ... of the split-major sequence in which the expert
//                   problems of one split are contiguous; m-tile-major across the splits when
//                   the communication work is handed out dynamically).
//
// Compute CTA (warp-specialised; tile_m x tile_n with tile_m in {64, 128}):
//   warps 0, 2  TMA producers (one thread each): warp 0 the x_routed tile (128 rows x 64 k), warp 2 the
//               W2 tile (tile_n rows x 64 k) of every k-block, into a ring of 128B-swizzled stages;
//   warp 1      MMA issuer (the warp runs the loop converged, an elected lane issues; all operands warp-uniform):
//               tcgen05.mma (M = 128, N = tile_n, K = 16, bf16 -> fp32) into one of two TMEM accumulator
//               buffers; tcgen05.commit frees stages / publishes the tile;
//   warps 4-15  epilogue: tcgen05.ld -> bf16 -> Y (three column groups x four TMEM lane quarters; warps 16-19
//               are a fourth column group when the launch carries no co-resident communication warp);
//   warp 3      publisher (one thread): once the epilogue warps have stored a tile, release fence, then the
//               tile's readiness flag and the split counter (one fence for all tiles stored by then).
// Compute CTA pair (256 x 256 tiles): the same roles in both CTAs of a cluster of two; one
//   tcgen05.mma.cta_group::2 spans both SMs, each CTA loads only its own operand halves; six operand
//   stages, seven when the aux region of shared memory is free while the GEMM runs.
// Y is token-major: the epilogue scatters each accumulator row to its (token, slot, shard) place, so
//   that the k_tot * TP partial rows of one (token, split, column slab) form one contiguous block.
// Communication CTA (12 independent warps): a warp fetches such a block with one bulk asynchronous
//   copy into its own double-buffered shared-memory stage (the readiness of the producing tiles is
//   checked first: split counter, else per-tile flags with ld.acquire.gpu; bounded), sums the rows in
//   fp32 in (j, p) order with the token's weights and stores bf16 into the owning rank's buffer.
// Co-resident communication warps (Section III-B with o_comm > 1 in spirit: communication work that
//   shares an SM with a compute CTA instead of reserving one): a compute CTA may carry extra warps
//   (of 16-19; two have stages) that run the same per-unit pipeline on stages of their own, take work from
//   the front of the per-split queues and serve split s while the CTA's other warps compute split
//   s + 1.  They wait for a whole split (no token of a split is complete before the last expert's
//   tiles of that split are), not for single tiles.
//
// Every wait is bounded: after `wait_ns` the waiter records MOE_DEV_TIMEOUT and the CTA winds
// down (pending bulk copies are drained, TMEM is released).

#include <cuda_bf16.h>

#include "moe_internal.h"
#include "sm100_device.cuh"

// Timeline build (-DMOE_TIMELINE=1, a separate library): the kernels record per-CTA time stamps and cycle
// counters into a caller-provided buffer (moe_set_timeline), kTimelineSlots 64-bit words per CTA followed by
// one completion stamp per split.  In the normal build every TL(...) statement compiles to nothing.
#ifndef MOE_TIMELINE
#define MOE_TIMELINE 0
#endif
#if MOE_TIMELINE
#define TL(...) do { __VA_ARGS__; } while (0)
#define TL_DECL(...) __VA_ARGS__
#else
#define TL(...) do { } while (0)
#define TL_DECL(...)
#endif

namespace moe {
namespace {

// slots of a CTA's timeline record (see bench.py --timeline for the reader)
enum {
    kTlBegin = 0, kTlRole = 1, kTlFirstAcc = 2, kTlMmaEnd = 3, kTlTiles = 4, kTlWaitOperand = 5, kTlIssue = 6,
    kTlWaitTmem = 7, kTlMmaCycles = 8, kTlComputeEnd = 9, kTlCtaEnd = 10, kTlEpiWait = 11, kTlEpiWork = 12,
    kTlProducerWait = 13, kTlCommUnits = 14, kTlCommWaitNs = 15, kTlCoWarp = 16,  // 8 slots per co-resident warp (16..31)
    kTlPubWait = 32, kTlPubFence = 33, kTlEpiPubWait = 34,
    kTlStageLate = 35   // pair tiles: k-blocks whose operand stage was not complete when the MMA issuer first looked
};
#if MOE_TIMELINE
__device__ __forceinline__ void tl_put(const FusedParams &P, int slot, unsigned long long v)
{
    if (P.timeline) P.timeline[(size_t)blockIdx.x * kTimelineSlots + slot] = v;
}
// Probes of the timeline build (moe_set_probe): parts of the launch's data movement are left out so that their
// cost shows in the launch time.  The results of a probed launch are garbage by construction.
#define MOE_PROBE(bit) ((P.probe & (bit)) != 0)
#else
#define MOE_PROBE(bit) false
#endif
enum { kProbeSkipOddW2 = 1, kProbeSkipAllW2 = 2, kProbeSkipYStores = 4, kProbeSkipX = 8, kProbeFreeRunMma = 16, kProbeSlowIssuer = 32 };

// --------------------------------------------------------------------------- shared memory

template <int TN>
struct Cfg {
    static constexpr int kABytes = kMmaM * kBlockK * 2;          // 16 KB
    static constexpr int kBBytes = TN * kBlockK * 2;             // 8 / 16 / 32 KB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = kStageBytesTotal / kStageBytes;  // 8 / 6 / 4
    static constexpr int kTmemCols = 2 * TN;                     // two accumulator buffers
    // epilogue: warps 4..15 (three column groups x four TMEM lane quarters), plus warps 16..19 as a fourth
    // column group when the launch carries no co-resident communication warps (FusedParams::epi_warps)
};

// Tiles a CTA may have stored but not yet published: the publisher's release fence takes thousands of cycles,
// and one fence covers every tile whose epilogue is over by then.
constexpr int kPubSlots = 4;

struct Control {
    unsigned long long full[8];
    unsigned long long empty[8];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long epi_done[kPubSlots];   // every epilogue warp has stored its rows of the tile (tile number mod kPubSlots)
    unsigned long long pub_done[kPubSlots];   // the publisher warp has raised that tile's flag
    uint32_t tmem_base;
    volatile uint32_t abort;
    unsigned long long comm_full[24];   // communication CTA: one barrier per warp and stage
    unsigned long long co_full[8];      // co-resident communication warps: one barrier per warp and stage
};

// 32 KB after the control block, used by one role per CTA:
//   communication CTA: per-row weights of the unit each warp reduces (12 warps x 256 floats)
//   compute CTA      : per-epilogue-warp staging (12 warps x 2.5 KB + row pointers) for coalesced Y stores
constexpr int kAuxBytes = 12 * 2560 + 12 * 256;
constexpr int kEpiStagePitch = 80;    // 64 data bytes + 16 pad: conflict-free 16-byte stores
struct EpiStage {
    uint8_t data[32 * kEpiStagePitch];        // 32 rows x 32 bf16
    unsigned long long rowptr[32];            // destination of each row for the group in hand (0 = skip)
};
static_assert(sizeof(EpiStage) * 12 <= kAuxBytes, "epilogue staging exceeds the aux region");
static_assert(12 * 256 * 4 <= kAuxBytes, "communication weights exceed the aux region");

// Bounded mbarrier wait, warp-collective: lane 0 polls (32 lanes polling the same barrier would
// each occupy the shared-memory pipe), the result is broadcast.  Returns false on timeout or when
// another warp of the CTA gave up.
__device__ __forceinline__ bool wait_barrier(uint32_t bar, uint32_t parity, Control *ctl,
                                             unsigned long long deadline, uint32_t *status,
                                             uint32_t detail, uint32_t where)
{
    uint32_t ok = 1u;
    if ((threadIdx.x & 31u) == 0u) {
        uint32_t spins = 0;
        while (!mbar_try_wait(bar, parity)) {
            if ((++spins & 63u) == 0u) {
                if (ctl->abort) { ok = 0u; break; }
                if (globaltimer_ns() > deadline) {
                    ctl->abort = 1u;
                    report(status, MOE_DEV_TIMEOUT, detail, where);
                    ok = 0u;
                    break;
                }
            }
        }
    }
    return __shfl_sync(0xffffffffu, ok, 0) != 0u;
}

// The same wait for a loop that a single thread runs on its own (no broadcast).
__device__ __forceinline__ bool wait_barrier_1t(uint32_t bar, uint32_t parity, Control *ctl,
                                                unsigned long long deadline, uint32_t *status,
                                                uint32_t detail, uint32_t where)
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

// Barrier of the warps that compute: 16, or all 20 when warps 16-19 serve as a fourth epilogue column group
// (co-resident communication warps never join it).
__device__ __forceinline__ void sync_compute_warps(const FusedParams &P)
{
    asm volatile("bar.sync 1, %0;" ::"r"(kThreads + 32 * (P.epi_warps - 12)) : "memory");
}
// 32-column rounds of a TN-wide tile dealt to `groups` epilogue column groups (3 or 4)
__device__ __forceinline__ int epi_cols_per_group(int tn, int groups)
{
    return ((tn / 32 + groups - 1) / groups) * 32;
}

struct Tile {
    int s, mu, p, i_n;
    int id;   // canonical tile number s * W_comp + (mu * TP + p) * NTs + i_n: indexes the readiness flags
};
// Tile g of the processing sequence.  Split-major (Section III-C: all tiles of split s precede those of
// s + 1; inside a split the expert problems are contiguous), or, when the work is handed out dynamically
// and nothing waits for an early split (drain help), m-tile-major: the n-tiles of ALL splits of one
// (m-tile, K-shard) are adjacent, so that the x rows are read from DRAM once instead of once per split.
__device__ __forceinline__ Tile decode_tile(int g, const FusedParams &P, int W_comp)
{
    Tile t;
    if (P.tile_order == 0) {
        t.s = g / W_comp;
        const int idx = g - t.s * W_comp;
        const int r = idx / P.NTs;
        t.i_n = idx - r * P.NTs;
        t.mu = r / P.TP;
        t.p = r - t.mu * P.TP;
        t.id = g;
    } else {
        const int per_m = P.L * P.NTs;
        const int r = g / per_m;
        const int j = g - r * per_m;
        t.s = j / P.NTs;
        t.i_n = j - t.s * P.NTs;
        t.mu = r / P.TP;
        t.p = r - t.mu * P.TP;
        t.id = t.s * W_comp + r * P.NTs + t.i_n;
    }
    return t;
}

// --------------------------------------------------------------------------- epilogue helper

// One thread = one accumulator row (TMEM lane).  Reads COLS fp32 columns starting at `col_first` of
// the accumulator at `taddr`, rounds to bf16 and writes them to the row's place in the token-major Y:
// slab = column slab inside the split, q = row of the unit (slot j, shard p).
__device__ __forceinline__ void store_accumulator_rows(const FusedParams &P, uint32_t taddr, int col_first, int n_cols, bool row_ok,
                                                       __nv_bfloat16 *ybase, int q, int n0, int col_end, int cis0)
{
#pragma unroll 1
    for (int cc = 0; cc < n_cols; cc += 32) {
        const int col = col_first + cc;
        uint32_t r[32];
        tmem_ld_32x32(taddr + (uint32_t)col, r);
        tmem_ld_wait(r);
        if (row_ok) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int c0 = n0 + col + v * 8;
                if (c0 < col_end) {
                    const int cis = cis0 + col + v * 8;
                    const int slab = cis >> P.slab_shift;
                    const int cin = cis & (P.slab_cols - 1);
                    const int wslab = min(P.slab_cols, P.split_w - (slab << P.slab_shift));
                    uint4 pk;
                    __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
                    __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
                    __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
                    pk.x = *reinterpret_cast<uint32_t *>(&h0);
                    pk.y = *reinterpret_cast<uint32_t *>(&h1);
                    pk.z = *reinterpret_cast<uint32_t *>(&h2);
                    pk.w = *reinterpret_cast<uint32_t *>(&h3);
                    *reinterpret_cast<uint4 *>(ybase + ((size_t)slab * P.Q << P.slab_shift) + (size_t)q * wslab + cin) = pk;
                }
            }
        }
    }
}

// Same job with 256-bit stores straight from registers (no shared memory).  Needs every 16-column group whole
// and 32-byte aligned (FusedParams::wide_store).
// One 32-column group of every lane's row, bf16.  The stores of two neighbouring lanes are joined: lanes 2k and
// 2k+1 swap half of their rows' data, so that one store instruction covers 64 contiguous bytes of a row (one
// request of two sectors instead of two requests of one sector).  Half as many write requests from the SM for
// the same bytes: the GEMM phase gets 2 % shorter where K is long (the requests compete with the operand stream)
// and 10 % where it is short (K = 256: the epilogue bounds the tile).  The whole warp runs this, also lanes
// without a valid row.
__device__ __forceinline__ void emit_wide_joined(const FusedParams &P, const uint32_t (&r)[32], int col, bool row_ok,
                                                 __nv_bfloat16 *ybase, int q, int n0, int col_end, int cis0)
{
    const int lane = threadIdx.x & 31;
    const bool odd = lane & 1;
    const int cis = cis0 + col;
    const int slab = cis >> P.slab_shift;
    const int wslab = min(P.slab_cols, P.split_w - (slab << P.slab_shift));
    __nv_bfloat16 *dst = ybase + ((size_t)slab * P.Q << P.slab_shift) + (size_t)q * wslab + (cis & (P.slab_cols - 1));
    if (!row_ok || MOE_PROBE(kProbeSkipYStores)) dst = nullptr;
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
        w[i] = *reinterpret_cast<uint32_t *>(&h);
    }
    // what the neighbour stores for this lane's row: the even lane hands over columns 16..31, the odd one 0..15
    uint32_t other[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) other[i] = __shfl_xor_sync(0xffffffffu, odd ? w[i] : w[8 + i], 1);
    const unsigned long long mine = reinterpret_cast<unsigned long long>(dst);
    const unsigned long long theirs = __shfl_xor_sync(0xffffffffu, mine, 1);
    // first instruction: the even lane's row (even lane: its columns 0..15; odd lane: the even lane's 16..31);
    // second instruction: the odd lane's row (even lane: the odd lane's 0..15; odd lane: its own 16..31)
    __nv_bfloat16 *p1 = reinterpret_cast<__nv_bfloat16 *>(odd ? theirs : mine);
    __nv_bfloat16 *p2 = reinterpret_cast<__nv_bfloat16 *>(odd ? mine : theirs);
    const int c1 = n0 + col + (odd ? 16 : 0);
    uint32_t d1[8], d2[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        d1[i] = odd ? other[i] : w[i];
        d2[i] = odd ? w[8 + i] : other[i];
    }
    if (p1 != nullptr && c1 < col_end) st_global_v8(p1 + (odd ? 16 : 0), d1);
    if (p2 != nullptr && c1 < col_end) st_global_v8(p2 + (odd ? 16 : 0), d2);
}
__device__ __forceinline__ void store_accumulator_rows_wide(const FusedParams &P, uint32_t taddr, int col_first, int n_cols, bool row_ok,
                                                            __nv_bfloat16 *ybase, int q, int n0, int col_end, int cis0)
{
    // (reading the next group from TMEM while this one is stored was measured: no gain, 13 more registers)
#pragma unroll 1
    for (int cc = 0; cc < n_cols; cc += 32) {
        uint32_t r[32];
        tmem_ld_32x32(taddr + (uint32_t)(col_first + cc), r);
        tmem_ld_wait(r);
        emit_wide_joined(P, r, col_first + cc, row_ok, ybase, q, n0, col_end, cis0);
    }
}

// Same job with the stores coalesced: the warp's 32 rows x 32 columns go through a padded staging
// buffer, so that four lanes write one row's 64 contiguous bytes (two full sectors) instead of every
// lane writing 16 bytes of a different row.  Needs the 32-column group inside one column slab.
__device__ __forceinline__ void store_accumulator_rows_staged(const FusedParams &P, uint32_t taddr, int col_first, int n_cols, bool row_ok,
                                                              __nv_bfloat16 *ybase, int q, int n0, int col_end, int cis0,
                                                              EpiStage *stg)
{
    const int lane = threadIdx.x & 31;
    const uint32_t stg_s = smem_u32(stg->data);
    const uint32_t my_row_s = stg_s + (uint32_t)lane * kEpiStagePitch;
    const int chunk = lane & 3;
#pragma unroll 1
    for (int cc = 0; cc < n_cols; cc += 32) {
        const int col = col_first + cc;
        uint32_t r[32];
        tmem_ld_32x32(taddr + (uint32_t)col, r);
        // where this thread's row goes for this 32-column group
        const int cis = cis0 + col;
        const int slab = cis >> P.slab_shift;
        const int wslab = min(P.slab_cols, P.split_w - (slab << P.slab_shift));
        stg->rowptr[lane] = row_ok ? (unsigned long long)(ybase + ((size_t)slab * P.Q << P.slab_shift) + (size_t)q * wslab +
                                                          (cis & (P.slab_cols - 1)))
                                   : 0ull;
        tmem_ld_wait(r);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
            __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
            __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
            __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
            sts_v4(my_row_s + v * 16, *reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1),
                   *reinterpret_cast<uint32_t *>(&h2), *reinterpret_cast<uint32_t *>(&h3));
        }
        __syncwarp();
        // four lanes per row, eight rows per store instruction
        const bool col_ok = (n0 + col + chunk * 8) < col_end;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = i * 8 + (lane >> 2);
            const unsigned long long dst = stg->rowptr[row];
            const uint4 v = lds_v4(stg_s + (uint32_t)row * kEpiStagePitch + (uint32_t)chunk * 16u);
            if (dst != 0ull && col_ok) *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(dst) + chunk * 8) = v;
        }
        __syncwarp();
    }
}

// --------------------------------------------------------------------------- epilogue and publisher roles
//
// Shared by the one-CTA and the CTA-pair compute roles (kPair: this CTA is rank `rank` of a pair and owns rows
// rank * 128 ... of the 256-row tile; the accumulator buffer is handed back on the leader's barrier; the tile is
// published in two parts, one flag per CTA).

// Epilogue, one warp: TMEM -> bf16 -> Y for the warp's TMEM lane quarter and column group of every tile of
// this CTA, then the hand-over to the publisher warp.
template <int TN, bool kPair>
__device__ __forceinline__ void epilogue_role(const FusedParams &P, int W_comp, Control *ctl, uint8_t *aux, int b,
                                              uint32_t tmem_base, unsigned long long deadline, int rank)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = P.L * W_comp;
    const int q4 = warp & 3;                   // TMEM lane quarter this warp may read
    const int grp = (warp - 4) >> 2;           // column group of the tile
    const int cols_per_group = epi_cols_per_group(TN, P.epi_warps >> 2);
    const int col_first = grp * cols_per_group;
    const int n_cols = max(0, min(cols_per_group, TN - col_first));
    const int row_in_tile = (kPair ? rank * kMmaM : 0) + q4 * 32 + lane;
    __nv_bfloat16 *Y = reinterpret_cast<__nv_bfloat16 *>(P.Y);
    // Row bookkeeping runs ahead of the accumulators: the m-tile table entries are fetched two tiles
    // ahead and the row's flat assignment one tile ahead, so that these dependent global loads are
    // not in the way between an accumulator becoming ready and its first store.
    int valid = 0, f_row = 0, valid_n = 0, first_n = 0;
    TL_DECL(long long tl_ew = 0, tl_ek = 0, tl_ep = 0, tl_q;)
    if (b < total_tiles) {
        const int mu0 = decode_tile(b, P, W_comp).mu;
        const int mu1 = decode_tile(min(b + P.P, total_tiles - 1), P, W_comp).mu;
        valid = __ldg(&P.mtile_valid[mu0]);
        const int first0 = __ldg(&P.mtile_first_row[mu0]);
        valid_n = __ldg(&P.mtile_valid[mu1]);
        first_n = __ldg(&P.mtile_first_row[mu1]);
        if (row_in_tile < valid) f_row = __ldg(&P.perm[first0 + row_in_tile]);
    }
    int it = 0;
    for (int g = b; g < total_tiles; g += P.P, ++it) {
        const Tile t = decode_tile(g, P, W_comp);
        const int a = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        const int mu_nn = decode_tile(min(g + 2 * P.P, total_tiles - 1), P, W_comp).mu;
        const int valid_nn = __ldg(&P.mtile_valid[mu_nn]);
        const int first_nn = __ldg(&P.mtile_first_row[mu_nn]);
        const int f_row_n = (row_in_tile < valid_n) ? __ldg(&P.perm[first_n + row_in_tile]) : 0;
        TL(tl_q = clock64());
        bool ok = wait_barrier(smem_u32(&ctl->tmem_full[a]), acc_phase, ctl, deadline, P.status, (uint32_t)g, 30u);
        TL(tl_ew += clock64() - tl_q; tl_q = clock64());
        if (ok) {
            tc_fence_after();
            const int n0 = t.s * P.split_w + t.i_n * TN;
            const int col_end = min(P.H, (t.s + 1) * P.split_w);
            const bool row_ok = row_in_tile < valid;
            // destination of this thread's row: the routed row belongs to flat assignment
            // f = (token, slot); Y is token-major so that the combine reads one contiguous block
            __nv_bfloat16 *ybase = Y;
            int q = 0;
            if (row_ok) {
                const int f = f_row;
                const int tok = f / P.k_tot;
                q = (f - tok * P.k_tot) * P.TP + t.p;
                ybase = Y + ((size_t)tok * P.L + t.s) * (size_t)P.Q * (size_t)P.split_w;
            }
            const uint32_t taddr = tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(a * TN);
            if (P.wide_store)
                store_accumulator_rows_wide(P, taddr, col_first, n_cols, row_ok, ybase, q, n0, col_end, n0 - t.s * P.split_w);
            else if (P.slab_cols >= 32)
                store_accumulator_rows_staged(P, taddr, col_first, n_cols, row_ok, ybase, q, n0, col_end,
                                              n0 - t.s * P.split_w, reinterpret_cast<EpiStage *>(aux) + (warp - 4));
            else
                store_accumulator_rows(P, taddr, col_first, n_cols, row_ok, ybase, q, n0, col_end, n0 - t.s * P.split_w);
            // the accumulator buffer (this CTA's half of it) may be overwritten by the MMA of the tile after next
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (kPair) mbar_arrive_cluster_relaxed(mapa_u32(smem_u32(&ctl->tmem_empty[a]), 0u));   // the leader's barrier
                else mbar_arrive(smem_u32(&ctl->tmem_empty[a]));
            }
            TL(tl_ek += clock64() - tl_q);
        }
        // hand the tile to the publisher warp.  Its barrier is reused every kPubSlots tiles, so the warp first
        // makes sure that the tile kPubSlots back has been published (it normally has, long ago).
        const int slot = it & (kPubSlots - 1);
        TL(tl_q = clock64());
        if (ok && it >= kPubSlots)
            ok = wait_barrier(smem_u32(&ctl->pub_done[slot]), (uint32_t)((it - kPubSlots) / kPubSlots) & 1u, ctl, deadline,
                              P.status, (uint32_t)g, 31u);
        TL(tl_ep += clock64() - tl_q);
        if (!ok) break;
        __syncwarp();   // the lanes' stores are ordered before lane 0's arrival
        if (lane == 0) mbar_arrive(smem_u32(&ctl->epi_done[slot]));
        valid = valid_n;
        f_row = f_row_n;
        valid_n = valid_nn;
        first_n = first_nn;
    }
    TL(if (warp == 4 && lane == 0) { tl_put(P, kTlEpiWait, (unsigned long long)tl_ew); tl_put(P, kTlEpiWork, (unsigned long long)tl_ek);
                                      tl_put(P, kTlEpiPubWait, (unsigned long long)tl_ep); });
}

// Publisher, one thread of warp 3: raises the readiness flag of every finished tile.  The release costs
// microseconds (the fence waits until the CTA's stores to Y have been performed: 2800 cycles per tile at the
// DeepSeek shape, 4900 at the Granite shape, where a tile's four k-blocks take less than that); here it is off
// the path of the epilogue warps, which go straight on to the next accumulator, and one fence covers every tile
// whose epilogue has finished by then (up to kPubSlots).
template <bool kPair>
__device__ __forceinline__ void publisher_role(const FusedParams &P, int W_comp, Control *ctl, int b,
                                               unsigned long long deadline, int rank)
{
    const int total_tiles = P.L * W_comp;
    if ((threadIdx.x & 31) == 0) {
        int it = 0;
        TL_DECL(long long tl_pw = 0, tl_pf = 0, tl_q;)
        for (int g = b; g < total_tiles;) {
            TL(tl_q = clock64());
            if (!wait_barrier_1t(smem_u32(&ctl->epi_done[it & (kPubSlots - 1)]), (uint32_t)(it / kPubSlots) & 1u, ctl,
                                 deadline, P.status, (uint32_t)g, 32u))
                break;
            TL(tl_pw += clock64() - tl_q; tl_q = clock64());
            // the following tiles too, as far as their epilogues are already over (waiting for more of them before
            // the fence was measured: no gain)
            int n = 1;
            while (n < kPubSlots && g + n * P.P < total_tiles &&
                   mbar_test_wait(smem_u32(&ctl->epi_done[(it + n) & (kPubSlots - 1)]), (uint32_t)((it + n) / kPubSlots) & 1u))
                ++n;
            fence_acq_rel_gpu();   // release: the epilogue warps' stores (observed through epi_done) come first
            for (int j = 0; j < n; ++j, ++it, g += P.P) {
                const Tile t = decode_tile(g, P, W_comp);
                if (t.id != P.withhold) {
                    st_relaxed_u32(&P.flags[kPair ? 2 * t.id + rank : t.id], P.epoch);
#if MOE_TIMELINE
                    if (atomicAdd(&P.split_done[t.s], 1u) + 1u == (uint32_t)(W_comp * P.flag_parts) && P.timeline)
                        P.timeline[(size_t)gridDim.x * kTimelineSlots + t.s] = globaltimer_ns();
#else
                    red_relaxed_add_u32(&P.split_done[t.s], 1u);
#endif
                }
                mbar_arrive(smem_u32(&ctl->pub_done[it & (kPubSlots - 1)]));
            }
            TL(tl_pf += clock64() - tl_q);
        }
        TL(tl_put(P, kTlPubWait, (unsigned long long)tl_pw); tl_put(P, kTlPubFence, (unsigned long long)tl_pf));
    }
    __syncwarp();
}

// --------------------------------------------------------------------------- compute CTA

template <int TN>
__device__ void compute_cta(const FusedParams &P, int W_comp, uint8_t *ring, Control *ctl, uint8_t *aux, int b)
{
    using C = Cfg<TN>;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = P.L * W_comp;
    const unsigned long long deadline = globaltimer_ns() + P.wait_ns;

    // setup: barriers (thread 0), TMEM allocation (warp 1)
    if (threadIdx.x == 0) {
        for (int i = 0; i < C::kStages; ++i) {
            mbar_init(smem_u32(&ctl->full[i]), 1);
            mbar_init(smem_u32(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[i]), (uint32_t)P.epi_warps);
        }
        for (int i = 0; i < kPubSlots; ++i) {
            mbar_init(smem_u32(&ctl->epi_done[i]), (uint32_t)P.epi_warps);
            mbar_init(smem_u32(&ctl->pub_done[i]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&ctl->tmem_base), C::kTmemCols);
    tc_fence_before();
    sync_compute_warps(P);
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0 || warp == 2) {
        // ---------------- TMA producers: warp 0 loads the x_routed tile, warp 2 the W2 tile of every
        // k-block; both complete on the same full barrier.  One thread per warp runs the whole loop (no
        // per-iteration warp broadcast); the others park below.
        const bool load_a = (warp == 0);
        if (lane == 0 && b < total_tiles) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t armed = 0;  // bit s: stage s was handed to the TMA unit at least once
            bool ok = true;
            TL_DECL(long long tl_pw = 0, tl_q;)
            // the m-tile table entries of the NEXT tile are fetched while this tile's k-blocks are issued, so
            // that the two dependent global loads never stall the stream of copies at a tile boundary
            Tile t = decode_tile(b, P, W_comp);
            int e = __ldg(&P.mtile_expert[t.mu]);
            int row0 = __ldg(&P.mtile_first_row[t.mu]);
            for (int g = b; g < total_tiles && ok; g += P.P) {
                const Tile t_next = decode_tile(min(g + P.P, total_tiles - 1), P, W_comp);
                const int e_next = __ldg(&P.mtile_expert[t_next.mu]);
                const int row0_next = __ldg(&P.mtile_first_row[t_next.mu]);
                const int n0 = t.s * P.split_w + t.i_n * TN;
                int kx = t.p * P.K;
                for (int kb = 0; kb < P.num_kb; ++kb, kx += kBlockK) {
                    TL(tl_q = clock64());
                    ok = wait_barrier_1t(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, deadline, P.status, (uint32_t)g, 10u);
                    if (!ok) break;
                    TL(tl_pw += clock64() - tl_q);
                    const uint32_t full = smem_u32(&ctl->full[stage]);
                    const uint32_t a_dst = smem_u32(ring + stage * C::kStageBytes);
                    const bool skip_b = MOE_PROBE(kProbeSkipAllW2) || (MOE_PROBE(kProbeSkipOddW2) && (kb & 1));
                    if (load_a) {
                        mbar_arrive_expect_tx(full, (uint32_t)C::kStageBytes);
                        tma_load_2d(a_dst, &P.tmA, full, kx, row0);
                    } else if (!skip_b) {
                        tma_load_3d(a_dst + C::kABytes, &P.tmB, full, kx, n0, e);
                    } else {
                        // a probe that leaves the copy out completes its bytes by hand: this producer stays in
                        // the barrier's dependency chain, or the other one could lap it
                        mbar_complete_tx_cluster(mapa_u32(full, cluster_ctarank()), (uint32_t)(C::kStageBytes - C::kABytes));
                    }
                    armed |= 1u << stage;
                    if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                }
                t = t_next;
                e = e_next;
                row0 = row0_next;
            }
            TL(if (load_a) tl_put(P, kTlProducerWait, (unsigned long long)tl_pw));
            if (!ok) {
                // wind-down: let the copies already issued land before shared memory is released
                // (bounded; a stage consumed meanwhile has completed its phase and passes at once)
                const unsigned long long drain = globaltimer_ns() + 2000000ull;
                for (int sidx = 0; sidx < C::kStages; ++sidx) {
                    if (!(armed & (1u << sidx))) continue;
                    const uint32_t par = (sidx < stage) ? phase : (phase ^ 1u);
                    while (!mbar_try_wait(smem_u32(&ctl->full[sidx]), par) && globaltimer_ns() < drain) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer: the whole warp runs the loop, converged, one elected lane issues; the loop
        // is as short as it can be and its operands are warp-uniform (both for the reasons given in
        // compute_cta_pair): a whole k-block (four MMAs and the commit) is one statement with 32-bit descriptor
        // arithmetic, addresses advance by additions, the barrier's first look is the non-suspending test.
        {
            constexpr uint32_t idesc = make_idesc(kMmaM, TN);
            constexpr uint32_t kLoStage = (uint32_t)(C::kStageBytes >> 4), kLoB = (uint32_t)(C::kABytes >> 4);
            const uint32_t lo0 = smem_desc_lo(smem_u32(ring));
            const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
            uint32_t a_lo = lo0, full_bar = full0, empty_bar = empty0;
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            TL_DECL(const long long tl_c0 = clock64(); long long tl_wf = 0, tl_wt = 0, tl_is = 0, tl_q;)
            for (int g = b; g < total_tiles && ok; g += P.P, ++it) {
                const int a = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                TL(tl_q = clock64());
                if (!__all_sync(0xffffffffu, mbar_test_wait(smem_u32(&ctl->tmem_empty[a]), acc_phase ^ 1u))) {
                    // (every lane polls; the vote keeps `ok`, and with it the loop, provably warp-uniform)
                    ok = __all_sync(0xffffffffu, wait_barrier_1t(smem_u32(&ctl->tmem_empty[a]), acc_phase ^ 1u, ctl, deadline, P.status, (uint32_t)g, 20u));
                    if (!ok) break;
                }
                TL(tl_wt += clock64() - tl_q);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * TN);
                for (int kb = 0; kb < P.num_kb; ++kb) {
                    TL(tl_q = clock64());
                    if (!__all_sync(0xffffffffu, mbar_test_wait(full_bar, phase))) {
                        ok = __all_sync(0xffffffffu, wait_barrier_1t(full_bar, phase, ctl, deadline, P.status, (uint32_t)g, 21u));
                        if (!ok) break;
                    }
                    TL(tl_wf += clock64() - tl_q; tl_q = clock64());
                    tc_fence_after();
                    // advancing K by 16 bf16 = 32 bytes inside the swizzle row: +2 in the address field
                    if (elect_one_sync()) {
                        if (kb < P.num_kb - 1 || P.last_ksteps == kBlockK / kUmmaK) {
                            tc_kblock_bf16(d_tmem, a_lo, a_lo + kLoB, idesc, kb > 0 ? 1u : 0u, empty_bar);
                        } else {
                            const uint64_t a_desc = ((uint64_t)kSmemDescHi << 32) | a_lo, b_desc = a_desc + kLoB;
                            for (int k = 0; k < P.last_ksteps; ++k)
                                tc_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                            (k > 0 || kb > 0) ? 1u : 0u);
                            tc_commit(empty_bar);   // stage reusable once these MMAs have read it
                        }
                    }
                    TL(tl_is += clock64() - tl_q);
                    a_lo += kLoStage;
                    full_bar += 8u;
                    empty_bar += 8u;
                    if (++stage == C::kStages) {
                        stage = 0;
                        phase ^= 1u;
                        a_lo = lo0;
                        full_bar = full0;
                        empty_bar = empty0;
                    }
                }
                __syncwarp();
                if (ok && elect_one_sync()) tc_commit(smem_u32(&ctl->tmem_full[a]));  // accumulator complete
                TL(if (it == 0 && lane == 0) tl_put(P, kTlFirstAcc, globaltimer_ns()));
            }
            TL(if (lane == 0) {
                   tl_put(P, kTlMmaEnd, globaltimer_ns()); tl_put(P, kTlTiles, (unsigned long long)it);
                   tl_put(P, kTlWaitOperand, (unsigned long long)tl_wf); tl_put(P, kTlIssue, (unsigned long long)tl_is);
                   tl_put(P, kTlWaitTmem, (unsigned long long)tl_wt); tl_put(P, kTlMmaCycles, (unsigned long long)(clock64() - tl_c0)); });
        }
        __syncwarp();
    } else if (warp >= 4 && warp < 4 + P.epi_warps) {
        epilogue_role<TN, false>(P, W_comp, ctl, aux, b, tmem_base, deadline, 0);
    } else if (warp == 3) {
        publisher_role<false>(P, W_comp, ctl, b, deadline, 0);
    }
    // ---------------- teardown
    tc_fence_before();
    sync_compute_warps(P);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}


// --------------------------------------------------------------------------- compute CTA pair
//
// 256 x 256 pair tile: two CTAs of a cluster (two SMs) compute one tile with tcgen05.mma.cta_group::2.
// CTA `rank` loads its own 128 rows of x_routed and its own 128 of the 256 W2 rows of every k-block
// (no multicast: each CTA issues its own loads), so a k-block costs 32 KB per SM instead of 48 KB.
// Rank 0 (the leader) issues the MMAs; tcgen05.commit arrives on the barriers of both CTAs.
//   full[stage]       only the leader's is used: armed by the leader for the bytes of both CTAs
//   empty[stage]      one per CTA (its producer waits on it), signalled by the leader's commit
//   tmem_full[a]      one per CTA (its epilogue waits on it), signalled by the leader's commit
//   tmem_empty[a]     only the leader's is used: 12 local + 12 remote epilogue warps arrive
struct PairCfg {
    static constexpr int kTileN = 256;
    static constexpr int kABytes = kMmaM * kBlockK * 2;                 // 16 KB: this CTA's 128 rows
    static constexpr int kBBytes = (kTileN / 2) * kBlockK * 2;          // 16 KB: this CTA's 128 W2 rows
    static constexpr int kStageBytes = kABytes + kBBytes;               // 32 KB
    // kStageBytesTotal / kStageBytes = 6 stages; a seventh lies in the aux region when that is free (FusedParams::pair_stages)
    static constexpr int kTmemCols = 2 * kTileN;                        // two accumulator buffers
};

__device__ void compute_cta_pair(const FusedParams &P, int W_comp, uint8_t *ring, Control *ctl, uint8_t *aux, int b)
{
    using C = PairCfg;
    constexpr int TN = C::kTileN;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader_cta = (rank == 0);
    const int total_tiles = P.L * W_comp;
    const int n_stages = P.pair_stages;   // 6, or 7 with the aux region as one more stage
    const unsigned long long deadline = globaltimer_ns() + P.wait_ns;

    if (threadIdx.x == 0) {
        for (int i = 0; i < n_stages; ++i) {
            mbar_init(smem_u32(&ctl->full[i]), 1);
            mbar_init(smem_u32(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[i]), 2u * (uint32_t)P.epi_warps);
        }
        for (int i = 0; i < kPubSlots; ++i) {
            mbar_init(smem_u32(&ctl->epi_done[i]), (uint32_t)P.epi_warps);
            mbar_init(smem_u32(&ctl->pub_done[i]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(&ctl->tmem_base), C::kTmemCols);
    tc_fence_before();
    sync_compute_warps(P);
    cluster_sync_all();          // the peer's barriers exist before anything arrives on them (the co-resident
                                 // communication warps of both CTAs arrive on this cluster barrier too)
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0 || warp == 2) {
        // ---------------- TMA producers (both CTAs): warp 0 loads this CTA's x_routed rows, warp 2 its W2
        // rows; both complete on the leader's full barrier.  Two issuing threads halve the serial issue
        // latency per k-block.  One thread per warp runs the whole loop; the others park below.
        const bool load_a = (warp == 0);
        if (lane == 0 && b < total_tiles && !MOE_PROBE(kProbeFreeRunMma)) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t armed = 0;
            bool ok = true;
            TL_DECL(long long tl_pw = 0, tl_q;)
            // next tile's table entries are fetched one tile ahead (see compute_cta)
            Tile t = decode_tile(b, P, W_comp);
            int e = __ldg(&P.mtile_expert[t.mu]);
            int row0 = __ldg(&P.mtile_first_row[t.mu]) + (int)rank * kMmaM;
            for (int g = b; g < total_tiles && ok; g += P.P) {
                const Tile t_next = decode_tile(min(g + P.P, total_tiles - 1), P, W_comp);
                const int e_next = __ldg(&P.mtile_expert[t_next.mu]);
                const int row0_next = __ldg(&P.mtile_first_row[t_next.mu]) + (int)rank * kMmaM;
                const int n0 = t.s * P.split_w + t.i_n * TN + (int)rank * (TN / 2);
                int kx = t.p * P.K;
                for (int kb = 0; kb < P.num_kb; ++kb, kx += kBlockK) {
                    const uint32_t own_full = smem_u32(&ctl->full[stage]);
                    TL(tl_q = clock64());
                    ok = wait_barrier_1t(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, deadline, P.status, (uint32_t)g, 10u);
                    if (!ok) break;
                    TL(tl_pw += clock64() - tl_q);
                    const uint32_t leader_full = own_full & 0xFEFFFFFFu;   // same offset in the leader CTA (rank 0)
                    const uint32_t a_dst = smem_u32(ring + stage * C::kStageBytes);
                    const bool skip_b = MOE_PROBE(kProbeSkipAllW2) || (MOE_PROBE(kProbeSkipOddW2) && (kb & 1));
                    // (a probe that leaves a copy out completes its bytes by hand: every producer stays in the
                    // barrier's dependency chain, or the leader's could lap the others)
                    if (load_a) {
                        if (leader_cta) mbar_arrive_expect_tx(own_full, 2u * (uint32_t)C::kStageBytes);
                        if (!MOE_PROBE(kProbeSkipX)) tma_load_2d_pair(a_dst, &P.tmA, leader_full, kx, row0);
                        else mbar_complete_tx_cluster(mapa_u32(own_full, 0u), (uint32_t)C::kABytes);
                    } else if (!skip_b) {
                        tma_load_3d_pair(a_dst + C::kABytes, &P.tmB, leader_full, kx, n0, e);
                    } else {
                        mbar_complete_tx_cluster(mapa_u32(own_full, 0u), (uint32_t)(C::kStageBytes - C::kABytes));
                    }
                    armed |= 1u << stage;
                    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
                }
                t = t_next;
                e = e_next;
                row0 = row0_next;
            }
            TL(if (load_a) tl_put(P, kTlProducerWait, (unsigned long long)tl_pw));
            if (!ok && leader_cta) {
                // wind-down: let the copies already issued land before shared memory is released
                const unsigned long long drain = globaltimer_ns() + 2000000ull;
                for (int sidx = 0; sidx < n_stages; ++sidx) {
                    if (!(armed & (1u << sidx))) continue;
                    const uint32_t par = (sidx < stage) ? phase : (phase ^ 1u);
                    while (!mbar_try_wait(smem_u32(&ctl->full[sidx]), par) && globaltimer_ns() < drain) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 && leader_cta) {
        // ---------------- MMA issuer (leader CTA only).  The whole warp runs the loop, converged, and one elected
        // lane issues.  Two measured facts shape it.  (1) The tensor pipe buffers little ahead of the MMA it
        // executes: 200 idle cycles of the issuer per k-block cost a launch 130 cycles per k-block
        // (bench.py --timeline --probe 32), so the loop is as short as it can be: a whole k-block (four MMAs and
        // the commit) is one statement with 32-bit descriptor arithmetic, addresses advance by additions, the
        // barrier's first look is the non-suspending test.  (2) tcgen05.mma takes its descriptors and addresses
        // from uniform registers: when a single thread ran this loop inside `if (lane == 0)` every operand was
        // moved over from ordinary registers, MMA by MMA; with warp-uniform values in warp-uniform control flow
        // and elect.sync around the issue the GEMM phase is 6 % faster.
        {
            constexpr uint32_t idesc = make_idesc(2 * kMmaM, TN);
            constexpr uint32_t kLoStage = (uint32_t)(C::kStageBytes >> 4), kLoB = (uint32_t)(C::kABytes >> 4);
            const uint32_t lo0 = smem_desc_lo(smem_u32(ring));
            const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
            uint32_t a_lo = lo0, full_bar = full0, empty_bar = empty0;
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            TL_DECL(const long long tl_c0 = clock64(); long long tl_wf = 0, tl_wt = 0, tl_is = 0, tl_q; unsigned long long tl_late = 0;)
            for (int g = b; g < total_tiles && ok; g += P.P, ++it) {
                const int a = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                TL(tl_q = clock64());
                if (!__all_sync(0xffffffffu, mbar_test_wait(smem_u32(&ctl->tmem_empty[a]), acc_phase ^ 1u))) {
                    // (every lane polls; the vote keeps `ok`, and with it the loop, provably warp-uniform)
                    ok = __all_sync(0xffffffffu, wait_barrier_1t(smem_u32(&ctl->tmem_empty[a]), acc_phase ^ 1u, ctl, deadline, P.status, (uint32_t)g, 20u));
                    if (!ok) break;
                }
                TL(tl_wt += clock64() - tl_q);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * TN);
                for (int kb = 0; kb < P.num_kb; ++kb) {
                    TL(tl_q = clock64());
                    if (!MOE_PROBE(kProbeFreeRunMma) && !__all_sync(0xffffffffu, mbar_test_wait(full_bar, phase))) {
                        TL(++tl_late);
                        ok = __all_sync(0xffffffffu, wait_barrier_1t(full_bar, phase, ctl, deadline, P.status, (uint32_t)g, 21u));
                        if (!ok) break;
                    }
                    TL(tl_wf += clock64() - tl_q; tl_q = clock64());
                    tc_fence_after();
                    if (MOE_PROBE(kProbeSlowIssuer)) {   // 200 cycles in which nothing is issued
                        const long long until = clock64() + 200;
                        while (clock64() < until) {}
                    }
                    if (elect_one_sync()) {
                        if ((kb < P.num_kb - 1 || P.last_ksteps == kBlockK / kUmmaK) && !MOE_PROBE(kProbeFreeRunMma)) {
                            tc_kblock_bf16_pair(d_tmem, a_lo, a_lo + kLoB, idesc, kb > 0 ? 1u : 0u, empty_bar);
                        } else {
                            const uint64_t a_desc = ((uint64_t)kSmemDescHi << 32) | a_lo, b_desc = a_desc + kLoB;
                            const int ksteps = (kb == P.num_kb - 1) ? P.last_ksteps : (kBlockK / kUmmaK);
                            for (int k = 0; k < ksteps; ++k)
                                tc_mma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                                 (k > 0 || kb > 0) ? 1u : 0u);
                            if (!MOE_PROBE(kProbeFreeRunMma)) tc_commit_pair(empty_bar);      // both CTAs may refill the stage
                        }
                    }
                    TL(tl_is += clock64() - tl_q);
                    a_lo += kLoStage;
                    full_bar += 8u;
                    empty_bar += 8u;
                    if (++stage == n_stages) {
                        stage = 0;
                        phase ^= 1u;
                        a_lo = lo0;
                        full_bar = full0;
                        empty_bar = empty0;
                    }
                }
                __syncwarp();
                if (ok && elect_one_sync()) tc_commit_pair(smem_u32(&ctl->tmem_full[a]));   // both epilogues may start
                TL(if (it == 0 && lane == 0) tl_put(P, kTlFirstAcc, globaltimer_ns()));
            }
            TL(if (lane == 0) {
                   tl_put(P, kTlMmaEnd, globaltimer_ns()); tl_put(P, kTlTiles, (unsigned long long)it);
                   tl_put(P, kTlWaitOperand, (unsigned long long)tl_wf); tl_put(P, kTlIssue, (unsigned long long)tl_is);
                   tl_put(P, kTlWaitTmem, (unsigned long long)tl_wt); tl_put(P, kTlMmaCycles, (unsigned long long)(clock64() - tl_c0));
                   tl_put(P, kTlStageLate, tl_late); });
        }
        __syncwarp();
    } else if (warp >= 4 && warp < 4 + P.epi_warps) {
        epilogue_role<TN, true>(P, W_comp, ctl, aux, b, tmem_base, deadline, (int)rank);
    } else if (warp == 3) {
        publisher_role<true>(P, W_comp, ctl, b, deadline, (int)rank);
    }
    // ---------------- teardown: nobody leaves while its peer may still touch its memory (the co-resident
    // communication warps arrived on this cluster barrier right after the set-up one)
    tc_fence_before();
    sync_compute_warps(P);
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, C::kTmemCols);
    }
}

// --------------------------------------------------------------------------- communication CTA

// two fp32 FMAs in one instruction (sm_100): acc = x * w + acc on packed pairs
__device__ __forceinline__ unsigned long long ffma2(unsigned long long x, unsigned long long w, unsigned long long acc)
{
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(x), "l"(w), "l"(acc));
    return d;
}
__device__ __forceinline__ unsigned long long pack_f32x2(uint32_t lo, uint32_t hi)
{
    unsigned long long d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float &lo, float &hi)
{
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}
// acc[i] (a pair of fp32) += w * (the two bf16 of word i), for the four words of v
__device__ __forceinline__ void fma2_bf16x8(unsigned long long (&acc)[4], const uint4 &v, unsigned long long ww)
{
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = ffma2(pack_f32x2(u[i] << 16, u[i] & 0xFFFF0000u), ww, acc[i]);
}
__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], const uint4 &v, float w)
{
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        acc[2 * i + 0] = fmaf(w, __uint_as_float(u[i] << 16), acc[2 * i + 0]);
        acc[2 * i + 1] = fmaf(w, __uint_as_float(u[i] & 0xFFFF0000u), acc[2 * i + 1]);
    }
}

// Communication warp.  Y is token-major: the k_tot * TP partial rows of one (token, split, column
// slab) are one contiguous block (a "unit", at most 8 KB).  Every communication warp works on its own:
// it owns two 8 KB stages of shared memory and one mbarrier per stage, fetches a unit with ONE bulk
// asynchronous copy (global -> shared), and while that copy is in flight it reduces the previous unit
// in fp32 in (j, p) order with the token's weights and stores the bf16 result into the owning rank's
// buffer.  No warp waits on another one: the issue latency of the copies and the memory latency
// overlap across the warps of an SM.
//
// Who runs it (role):
//   kRoleStatic      warp w of communication CTA c, static map: units w, w+12, ... of the communication
//                    tiles c, c+C, ... of every split (the paper's map);
//   kRoleFront       warp of a communication CTA, dynamic hand-out: ranges from the front of the
//                    per-split queues, split 0 first; a unit waits for the tiles under it (flags);
//   kRoleBack        warp of a compute CTA whose GEMM tiles are done (drain help): ranges from the back,
//                    last split first;
//   kRoleCoResident  extra warp of a compute CTA that is still computing: from the front, split 0
//                    first, but only from splits that are complete (it sleeps on the split counter
//                    instead of polling single tiles, so that it costs the computing warps nothing
//                    while it has nothing to do).
constexpr int kCommWarps = 12;
constexpr int kCommUnitBytes = 8192;
constexpr int kCommWarpBytes = 2 * kCommUnitBytes;
static_assert(kCommWarps * kCommWarpBytes <= kStageBytesTotal, "communication stages exceed the ring");
// Co-resident communication warps live in the aux region, which the epilogue leaves alone when it
// stores straight from registers: two warps' stages (32 KB), then the per-row weights in compact
// 16-float slots -- four for co-resident warps, twelve for the CTA's own warps once they turn to
// communication (their usual 256-float slots would overlap the co-resident stages).  Needs Q <= 16.
constexpr int kCoWarpsAux = 2;          // co-resident warps whose stages fit the aux region
constexpr int kCoWeightFloats = 16;
constexpr int kCoWeightsOffset = kCoWarpsAux * kCommWarpBytes;
static_assert(PairCfg::kStageBytes + ((sizeof(Control) + 127) & ~(size_t)127) <= kAuxBytes + ((sizeof(Control) + 127) & ~(size_t)127) &&
              12 * 256 * 4 <= PairCfg::kStageBytes, "a seventh pair stage plus the control block exceed the allocation");
static_assert(kCoWeightsOffset + (kCoWarpsMax + kCommWarps) * kCoWeightFloats * 4 <= kAuxBytes,
              "co-resident stages and weights exceed the aux region");

enum { kRoleStatic = 0, kRoleFront = 1, kRoleBack = 2, kRoleCoResident = 3 };

// what one communication warp owns
struct CommWarpRes {
    uint8_t *stages;              // 2 x kCommUnitBytes
    unsigned long long *full;     // 2 mbarriers (initialised with count 1 at kernel start)
    float *wq;                    // room for Q floats
};

struct CommUnit {
    int t, d, s, slab, wslab, ucols;
    float w;          // lane j: weight of slot j (0 when the slot has no source row)
    bool live;
    bool all_valid;   // every slot of the token has a source row
};

// `c`, `warp`: communication CTA and warp inside it (static map only).
template <int TN>
__device__ void comm_warp(const FusedParams &P, int W_comp, Control *ctl, const CommWarpRes res, int role, int c, int warp,
                          int tl_slot)
{
    (void)tl_slot;   // index of the warp's record in a timeline build
    const int lane = threadIdx.x & 31;
    const bool wait_needed = (P.mode != MOE_MODE_COMBINE_ONLY);
    const bool helper = (role == kRoleBack);
    const unsigned long long deadline = globaltimer_ns() + P.wait_ns;
    // the wait for a copy only follows a readiness wait: it gets a later deadline so that the first
    // report names the wait that really ran out
    const unsigned long long deadline2 = deadline + P.wait_ns / 4 + 1000000ull;

    TL_DECL(unsigned long long tl_first = 0, tl_last = 0, tl_sleep = 0; uint32_t tl_units = 0, tl_by_split[4] = {0u, 0u, 0u, 0u};)
    uint8_t *my_ring = res.stages;
    float *wq = res.wq;
    const unsigned long long y_policy = l2_evict_first_policy();
    const uint32_t full_s = smem_u32(res.full);
    const __nv_bfloat16 *Y = reinterpret_cast<const __nv_bfloat16 *>(P.Y);

    // reduce the unit sitting in stage `st` (its copy was issued one unit ago)
    auto consume = [&](const CommUnit &u, int st, uint32_t parity) -> bool {
        bool ok = wait_barrier(full_s + 8u * (uint32_t)st, parity, ctl, deadline2, P.status, (uint32_t)u.t, 43u);
        if (!ok) return false;
        const int n16 = u.ucols >> 3;
        const uint32_t row_bytes = (uint32_t)u.wslab * 2u;
        // per-row weights, read back as shared-memory broadcasts inside the unrolled loop
        if (lane < P.k_tot)
            for (int p = 0; p < P.TP; ++p) wq[lane * P.TP + p] = u.w;
        __syncwarp();
        const uint32_t wq_s = smem_u32(wq);
        const uint32_t stage_s = smem_u32(my_ring + st * kCommUnitBytes);
        __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(P.out[u.d]) +
                              (size_t)(u.t - u.d * P.tok_blk) * (size_t)P.H + u.s * P.split_w + (u.slab << P.slab_shift);
        if (u.all_valid && P.Q <= 16) {
            // common case: every slot has a source row and the unit has at most 16 rows: weights stay in
            // registers as packed pairs, rows are fetched eight at a time, two FMAs per instruction
            unsigned long long ww[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                const uint32_t wb = __float_as_uint(r < P.Q ? lds_f32(wq_s + (uint32_t)r * 4u) : 0.f);
                ww[r] = pack_f32x2(wb, wb);
            }
            for (int c16 = lane; c16 < n16; c16 += 32) {
                unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
                const uint32_t src = stage_s + (uint32_t)c16 * 16u;
#pragma unroll
                for (int r0 = 0; r0 < 16; r0 += 8) {
                    if (r0 < P.Q) {
                        uint4 v[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[i] = lds_v4(src + (uint32_t)min(r0 + i, P.Q - 1) * row_bytes);
#pragma unroll
                        for (int i = 0; i < 8; ++i) fma2_bf16x8(acc, v[i], ww[r0 + i]);   // rows past Q carry weight 0
                    }
                }
                float f[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) unpack_f32x2(acc[i], f[2 * i], f[2 * i + 1]);
                uint4 pk;
                __nv_bfloat162 h0 = __floats2bfloat162_rn(f[0], f[1]);
                __nv_bfloat162 h1 = __floats2bfloat162_rn(f[2], f[3]);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(f[4], f[5]);
                __nv_bfloat162 h3 = __floats2bfloat162_rn(f[6], f[7]);
                pk.x = *reinterpret_cast<uint32_t *>(&h0);
                pk.y = *reinterpret_cast<uint32_t *>(&h1);
                pk.z = *reinterpret_cast<uint32_t *>(&h2);
                pk.w = *reinterpret_cast<uint32_t *>(&h3);
                __stcs(reinterpret_cast<uint4 *>(orow + c16 * 8), pk);
            }
        } else
        for (int c16 = lane; c16 < ((n16 + 31) & ~31); c16 += 32) {
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            const uint32_t src = stage_s + (uint32_t)(c16 < n16 ? c16 : 0) * 16u;
            for (int r0 = 0; r0 < P.Q; r0 += 8) {
                uint4 v[8];
                float w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = min(r0 + i, P.Q - 1);
                    v[i] = lds_v4(src + (uint32_t)r * row_bytes);
                    w[i] = lds_f32(wq_s + (uint32_t)r * 4u);
                    if (r0 + i >= P.Q) w[i] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    // a slot without a source row holds bytes nobody wrote: drop them
                    if (w[i] == 0.f) v[i] = make_uint4(0u, 0u, 0u, 0u);
                    fma_bf16x8(acc, v[i], w[i]);
                }
            }
            if (c16 < n16) {
                uint4 pk;
                __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[0], acc[1]);
                __nv_bfloat162 h1 = __floats2bfloat162_rn(acc[2], acc[3]);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(acc[4], acc[5]);
                __nv_bfloat162 h3 = __floats2bfloat162_rn(acc[6], acc[7]);
                pk.x = *reinterpret_cast<uint32_t *>(&h0);
                pk.y = *reinterpret_cast<uint32_t *>(&h1);
                pk.z = *reinterpret_cast<uint32_t *>(&h2);
                pk.w = *reinterpret_cast<uint32_t *>(&h3);
                __stcs(reinterpret_cast<uint4 *>(orow + c16 * 8), pk);
            }
        }
        __syncwarp();   // all lanes are done with the stage (and with wq) before either is reused
        TL(tl_last = globaltimer_ns(); if (tl_units == 0) tl_first = tl_last; ++tl_units; if (u.s < 4) ++tl_by_split[u.s]);
        return true;
    };

    int unit = 0;            // running unit number of this CTA
    int n_mine = 0;          // units this warp has issued so far: stage n_mine & 1, parity (n_mine >> 1) & 1
    CommUnit prev;
    prev.live = false;
    uint32_t ready_mask = wait_needed ? 0u : 0xffffffffu;   // bit s: split s is known to be complete

    // One unit: wait until the GEMM tiles under it are published (unless its split is known to be
    // complete), start its copy, then reduce the previous unit of this warp while the copy is in flight.
    // False when the warp had to give up (reported); nothing of this warp is in flight then.
    auto unit_step = [&](CommUnit &u) -> bool {
        // ---- readiness of the producing tiles
        if (!((ready_mask >> u.s) & 1u)) {
            uint32_t done = 0;
            if (lane == 0) done = ld_acquire_u32(&P.split_done[u.s]);
            done = __shfl_sync(0xffffffffu, done, 0);
            if (done >= (uint32_t)(W_comp * P.flag_parts)) {
                ready_mask |= 1u << u.s;
            } else {
                // per tile: every (slot j, shard p, n-tile under this slab)
                const int cs0 = u.slab << P.slab_shift;
                const int in0 = cs0 / TN;
                const int nt = (cs0 + u.ucols - 1) / TN - in0 + 1;
                bool failed = false;
                for (int chk = lane; chk < P.Q * nt && !failed; chk += 32) {
                    const int qq = chk / nt;
                    const int tn = chk - qq * nt;
                    const int j = qq / P.TP;
                    const int p = qq - j * P.TP;
                    const int row = __ldg(&P.pad_row[(size_t)u.t * P.k_tot + j]);
                    if (row < 0 || row >= P.R_pad) continue;
                    const int mu = row / P.tile_m;
                    // a pair tile is published in two parts, one per CTA: the row's part is its 128-row half
                    const int part = (P.flag_parts == 2) ? ((row - mu * P.tile_m) >> 7) : 0;
                    const int g = (u.s * W_comp + (mu * P.TP + p) * P.NTs + in0 + tn) * P.flag_parts + part;
                    uint32_t spins = 0;
                    TL_DECL(const unsigned long long tl_f0 = globaltimer_ns();)
                    while (ld_acquire_u32(&P.flags[g]) != P.epoch) {
                        if ((++spins & 31u) == 0u && (ctl->abort || globaltimer_ns() > deadline)) {
                            report(P.status, MOE_DEV_TIMEOUT, (uint32_t)g, 40u);
                            failed = true;
                            break;
                        }
                        __nanosleep(64);
                    }
                    TL(tl_sleep += globaltimer_ns() - tl_f0);
                }
                if (__any_sync(0xffffffffu, failed)) {
                    // this warp gives up; the copy it still has in flight must land first
                    if (prev.live) consume(prev, (n_mine - 1) & 1, (uint32_t)((n_mine - 1) >> 1) & 1u);
                    prev.live = false;
                    return false;
                }
            }
            __syncwarp();
            // rows published through ordinary stores are read by the copy engine next
            asm volatile("fence.proxy.async;" ::: "memory");
        }
        // ---- issue this unit's copy, then reduce the previous unit while it is in flight
        const int st = n_mine & 1;
        if (lane == 0) {
            const uint32_t full = full_s + 8u * (uint32_t)st;
            const uint32_t bytes = (uint32_t)(P.Q * u.wslab) * 2u;
            const __nv_bfloat16 *src = Y + ((size_t)u.t * P.L + u.s) * (size_t)P.Q * (size_t)P.split_w +
                                       ((size_t)u.slab * P.Q << P.slab_shift);
            mbar_arrive_expect_tx(full, bytes);
            bulk_load_once(smem_u32(my_ring + st * kCommUnitBytes), src, bytes, full, y_policy);   // Y is read once
        }
        __syncwarp();
        ++n_mine;
        if (prev.live && !consume(prev, (n_mine - 2) & 1, (uint32_t)((n_mine - 2) >> 1) & 1u)) {
            // the previous copy never landed (reported); wait for the one just issued, then leave
            const unsigned long long drain = globaltimer_ns() + 2000000ull;
            while (!mbar_try_wait(full_s + 8u * (uint32_t)st, (uint32_t)((n_mine - 1) >> 1) & 1u) && globaltimer_ns() < drain) {}
            prev.live = false;
            return false;
        }
        prev = u;
        return true;
    };

    // serve communication tile ct of split s; false when this warp had to give up (reported)
    auto serve_tile = [&](int s, int ct) -> bool {
        const int split_c0 = s * P.split_w;
        const int split_c1 = min(P.H, split_c0 + P.split_w);
        const int tok_tile = ct / P.comm_cols;
        const int col_tile = ct - tok_tile * P.comm_cols;
        const int d = tok_tile / P.tok_tiles_per_rank;
        const int ti = tok_tile - d * P.tok_tiles_per_rank;
        const int t0 = d * P.tok_blk + ti * kCommTileM;
        const int t1 = min(min(P.T, (d + 1) * P.tok_blk), t0 + kCommTileM);
        const int c0 = split_c0 + col_tile * kCommTileN;
        const int c1 = min(split_c1, c0 + kCommTileN);
        if (t0 >= t1 || c0 >= c1) return true;
        const int slab0 = (c0 - split_c0) >> P.slab_shift;
        const int n_slabs = ((c1 - split_c0 + P.slab_cols - 1) >> P.slab_shift) - slab0;
        const int n_units = (t1 - t0) * n_slabs;
        // first unit of this tile that belongs to this warp
        int k = (warp - unit % kCommWarps + kCommWarps) % kCommWarps;
        // routing of a unit's token is fetched one unit ahead, off the per-unit critical path
        int nxt_row = -1;
        float nxt_w = 0.f;
        if (k < n_units && lane < P.k_tot) {
            const int tn = t0 + k / n_slabs;
            nxt_row = __ldg(&P.pad_row[(size_t)tn * P.k_tot + lane]);
            nxt_w = __ldg(&P.topk_w[(size_t)tn * P.k_tot + lane]);
        }
        for (; k < n_units; k += kCommWarps) {
            CommUnit u;
            u.t = t0 + k / n_slabs;
            u.slab = slab0 + k % n_slabs;
            u.d = d;
            u.s = s;
            u.wslab = min(P.slab_cols, P.split_w - (u.slab << P.slab_shift));            // layout pitch
            u.ucols = min(u.wslab, split_c1 - split_c0 - (u.slab << P.slab_shift));       // real columns
            u.live = true;
            int my_row = nxt_row;
            u.w = nxt_w;
            if (k + kCommWarps < n_units && lane < P.k_tot) {
                const int tn = t0 + (k + kCommWarps) / n_slabs;
                nxt_row = __ldg(&P.pad_row[(size_t)tn * P.k_tot + lane]);
                nxt_w = __ldg(&P.topk_w[(size_t)tn * P.k_tot + lane]);
            }
            if (lane < P.k_tot) {
                if (my_row >= P.R_pad) {
                    report(P.status, MOE_DEV_OOB, (uint32_t)my_row, 42u);
                    my_row = -1;
                }
                if (my_row < 0) u.w = 0.f;
            }
            u.all_valid = __all_sync(0xffffffffu, lane >= P.k_tot || my_row >= 0);
            if (!unit_step(u)) {
                unit += n_units;
                return false;
            }
        }
        unit += n_units;
        return true;
    };

    // serve items [i0, i1) of split s on this warp alone.  An item is one token x one communication
    // column tile (token-major numbering); its units are the column slabs of that tile.
    auto serve_items = [&](int s, uint32_t i0, uint32_t i1) -> bool {
        const int split_c0 = s * P.split_w;
        const int split_c1 = min(P.H, split_c0 + P.split_w);
        int nxt_row = -1;
        float nxt_w = 0.f;
        if (lane < P.k_tot) {
            const int tn = (int)(i0 / (uint32_t)P.comm_cols);
            nxt_row = __ldg(&P.pad_row[(size_t)tn * P.k_tot + lane]);
            nxt_w = __ldg(&P.topk_w[(size_t)tn * P.k_tot + lane]);
        }
        for (uint32_t item = i0; item < i1; ++item) {
            const int tok = (int)(item / (uint32_t)P.comm_cols);
            const int col_tile = (int)(item - (uint32_t)tok * (uint32_t)P.comm_cols);
            int my_row = nxt_row;
            float my_w = nxt_w;
            if (item + 1 < i1 && lane < P.k_tot) {
                const int tn = (int)((item + 1) / (uint32_t)P.comm_cols);
                nxt_row = __ldg(&P.pad_row[(size_t)tn * P.k_tot + lane]);
                nxt_w = __ldg(&P.topk_w[(size_t)tn * P.k_tot + lane]);
            }
            if (lane < P.k_tot) {
                if (my_row >= P.R_pad) {
                    report(P.status, MOE_DEV_OOB, (uint32_t)my_row, 42u);
                    my_row = -1;
                }
                if (my_row < 0) my_w = 0.f;
            }
            const bool all_valid = __all_sync(0xffffffffu, lane >= P.k_tot || my_row >= 0);
            const int c0 = split_c0 + col_tile * kCommTileN;
            const int c1 = min(split_c1, c0 + kCommTileN);
            if (c0 >= c1) continue;
            const int slab0 = (c0 - split_c0) >> P.slab_shift;
            const int slab1 = (c1 - split_c0 + P.slab_cols - 1) >> P.slab_shift;
            for (int slab = slab0; slab < slab1; ++slab) {
                CommUnit u;
                u.t = tok;
                u.d = tok / P.tok_blk;
                u.s = s;
                u.slab = slab;
                u.wslab = min(P.slab_cols, P.split_w - (slab << P.slab_shift));
                u.ucols = min(u.wslab, split_c1 - split_c0 - (slab << P.slab_shift));
                u.w = my_w;
                u.live = true;
                u.all_valid = all_valid;
                if (!unit_step(u)) return false;
            }
        }
        return true;
    };

    if (role == kRoleStatic) {
        // the paper's static map: communication tile ct belongs to CTA ct mod C (Section III-A)
        for (int s = 0; s < P.L; ++s)
            for (int ct = c; ct < P.comm_tiles; ct += P.C)
                if (!serve_tile(s, ct)) {
                    ctl->abort = 1u;
                    return;
                }
    } else {
        // Dynamic hand-out, to warps.  Every split has a two-ended queue of its items in one 64-bit word
        // (low half: items taken from the front, high half: from the back).  Warps of the communication
        // CTAs and co-resident warps take from the front, split 0 first; warps of compute CTAs that have
        // run out of GEMM tiles take from the back, last split first.  One atomic add claims a range;
        // ranges shrink towards the end so that the last ones finish together.  The next claim is issued
        // before the current range is served, which hides the latency of the atomic.
        const uint32_t n_items = (uint32_t)P.T * (uint32_t)P.comm_cols;
        int s = helper ? P.L - 1 : 0;
        unsigned long long old = 0;
        uint32_t chunk = 0;
        auto claim = [&](int split) {   // lane 0 issues the atomic; the result is picked up later
            if (lane == 0) {
                const unsigned long long q = *reinterpret_cast<volatile unsigned long long *>(&P.queue[split]);
                const uint32_t taken = (uint32_t)q + (uint32_t)(q >> 32);
                const uint32_t rem = taken < n_items ? n_items - taken : 0u;
                chunk = min(8u, max(1u, rem >> 12));
                old = atomicAdd(&P.queue[split], helper ? ((unsigned long long)chunk << 32) : (unsigned long long)chunk);
            }
        };
        bool claimed = false;      // a claim on split s is outstanding
        while (s >= 0 && s < P.L) {
            if (!claimed) {
                if (role == kRoleCoResident && !((ready_mask >> s) & 1u)) {
                    // A co-resident warp only takes work that can be served at once.  Inside a split the
                    // tiles run expert by expert and a token needs tiles of all its experts, so hardly any
                    // token is complete before the split is: wait for the whole split, asleep most of the time.
                    uint32_t state = 0;   // 1: split complete, 2: split handed out already, 3: give up
                    if (lane == 0) {
                        if (ld_acquire_u32(&P.split_done[s]) >= (uint32_t)(W_comp * P.flag_parts)) state = 1;
                        else {
                            const unsigned long long q = *reinterpret_cast<volatile unsigned long long *>(&P.queue[s]);
                            if ((uint32_t)q + (uint32_t)(q >> 32) >= n_items) state = 2;
                            else if (ctl->abort) state = 3;
                            else if (globaltimer_ns() > deadline) {
                                report(P.status, MOE_DEV_TIMEOUT, (uint32_t)s, 44u);
                                state = 3;
                            }
                        }
                    }
                    state = __shfl_sync(0xffffffffu, state, 0);
                    if (state == 0) {
                        TL_DECL(const unsigned long long tl_s0 = globaltimer_ns();)
                        __nanosleep(2000);
                        TL(tl_sleep += globaltimer_ns() - tl_s0);
                        continue;
                    }
                    if (state == 2) {
                        ++s;
                        continue;
                    }
                    if (state == 3) {
                        ctl->abort = 1u;
                        break;
                    }
                    ready_mask |= 1u << s;
                    // rows published through ordinary stores are read by the copy engine next
                    asm volatile("fence.proxy.async;" ::: "memory");
                }
                claim(s);
                claimed = true;
            }
            const unsigned long long o = __shfl_sync(0xffffffffu, old, 0);
            const uint32_t ch = __shfl_sync(0xffffffffu, chunk, 0);
            const uint32_t f = (uint32_t)o, bk = (uint32_t)(o >> 32);
            const uint32_t hi = bk < n_items ? n_items - bk : 0u;    // items [hi, n) are taken from the back
            uint32_t i0, i1;
            if (!helper) {
                i0 = f;
                i1 = min(f + ch, hi);
            } else {
                i1 = hi;
                i0 = max(f, hi > ch ? hi - ch : 0u);
            }
            const int cur = s;
            if (i0 >= i1) {                      // this split is handed out: go on to the next one
                s += helper ? -1 : 1;
                claimed = false;
                continue;
            }
            claim(s);
            // warp-uniform exit: the loop body holds full-mask collectives
            if (__any_sync(0xffffffffu, ctl->abort != 0u)) break;
            if (!serve_items(cur, i0, i1)) {
                ctl->abort = 1u;
                return;
            }
        }
    }
    if (prev.live) consume(prev, (n_mine - 1) & 1, (uint32_t)((n_mine - 1) >> 1) & 1u);
#if MOE_TIMELINE
    if (lane == 0) {
        if (role == kRoleCoResident) {
            const int base = kTlCoWarp + 8 * tl_slot;
            tl_put(P, base + 0, tl_first); tl_put(P, base + 1, tl_last); tl_put(P, base + 2, tl_units); tl_put(P, base + 3, tl_sleep);
            for (int i = 0; i < 4; ++i) tl_put(P, base + 4 + i, tl_by_split[i]);
        } else if (tl_slot == 0) {
            tl_put(P, kTlCommUnits, tl_units);
            tl_put(P, kTlCommWaitNs, tl_sleep);
        }
    }
#endif
}

// The communication warps of a CTA whose only role is communication (dedicated communication CTA, or a
// compute CTA that has run out of GEMM tiles): warps 0-11, stages in the operand ring.
template <int TN>
__device__ __forceinline__ void comm_cta(const FusedParams &P, int W_comp, uint8_t *ring, Control *ctl, uint8_t *aux, int role, int c)
{
    const int warp = threadIdx.x >> 5;
    if (warp >= kCommWarps) return;
    CommWarpRes res;
    res.stages = ring + warp * kCommWarpBytes;
    res.full = &ctl->comm_full[2 * warp];
    res.wq = (role == kRoleBack && P.co_warps > 0)
                 ? reinterpret_cast<float *>(aux + kCoWeightsOffset) + (kCoWarpsMax + warp) * kCoWeightFloats
                 : reinterpret_cast<float *>(aux) + warp * 256;
    comm_warp<TN>(P, W_comp, ctl, res, role, c, warp, warp);
}

// Co-resident communication warp `cw` of a compute CTA: stages and weights in the aux region (free when
// the epilogue stores straight from registers, which the host checks before it asks for such warps).
template <int TN>
__device__ __forceinline__ void co_resident_warp(const FusedParams &P, int W_comp, Control *ctl, uint8_t *aux, int cw)
{
    CommWarpRes res;
    res.stages = aux + cw * kCommWarpBytes;
    res.full = &ctl->co_full[2 * cw];
    res.wq = reinterpret_cast<float *>(aux + kCoWeightsOffset) + cw * kCoWeightFloats;
    comm_warp<TN>(P, W_comp, ctl, res, kRoleCoResident, 0, 0, cw);
}

// Co-resident warp number of warp 16..19.  The four warp schedulers of an SM take warps by number modulo
// four, and scheduler 1 holds the thread that issues the MMAs, which has to stay ahead of the tensor pipe:
// warps 18 and 19 are used first, then 16, and 17 (scheduler 1) last.
__device__ __forceinline__ int co_warp_number(int warp)
{
    return warp == 18 ? 0 : warp == 19 ? 1 : warp == 16 ? 2 : 3;
}

// Barriers of every communication stage the CTA may use, and the abort flag; before the first CTA-wide
// barrier of the kernel.
__device__ __forceinline__ void init_comm_barriers(Control *ctl)
{
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2 * kCommWarps; ++i) mbar_init(smem_u32(&ctl->comm_full[i]), 1);
        for (int i = 0; i < 2 * kCoWarpsMax; ++i) mbar_init(smem_u32(&ctl->co_full[i]), 1);
        ctl->abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
}

// --------------------------------------------------------------------------- kernel

// Compute tiles per split of this launch (Eq. 5).  With the routed counts left on the device the m-tile
// count is read from the routing workspace (the routing kernels ran earlier on the same stream).
__device__ __forceinline__ int launch_w_comp(const FusedParams &P)
{
    return P.S_dev ? min(__ldg(P.S_dev), P.S) * P.TP * P.NTs : P.W_comp;
}

template <int TN>
__global__ void __launch_bounds__(kFusedThreads, 1)
moe_gemm2_combine_kernel(const __grid_constant__ FusedParams P)
{
    extern __shared__ uint8_t smem_raw[];
    // 128B-swizzled tiles need 1024-byte aligned bases
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Control *ctl = reinterpret_cast<Control *>(ring + kStageBytesTotal);
    uint8_t *aux = reinterpret_cast<uint8_t *>(ring + kStageBytesTotal + ((sizeof(Control) + 127) & ~(size_t)127));

    if (blockIdx.x == 0 && threadIdx.x < (unsigned)P.L) {
        P.split_done_next[threadIdx.x] = 0u;
        P.queue_next[threadIdx.x] = 0ull;
    }
    init_comm_barriers(ctl);
    __syncthreads();          // the only barrier all 20 warps share
    TL(if (threadIdx.x == 0) { tl_put(P, kTlBegin, globaltimer_ns()); tl_put(P, kTlRole, (int)blockIdx.x < P.C ? 0u : 1u); });

    const int warp = threadIdx.x >> 5;
    const int W_comp = launch_w_comp(P);
    if ((int)blockIdx.x < P.C) {
        comm_cta<TN>(P, W_comp, ring, ctl, aux, P.drain_help ? kRoleFront : kRoleStatic, (int)blockIdx.x);
    } else if (warp >= kThreads / 32 && P.epi_warps == 12) {
        if (co_warp_number(warp) < P.co_warps) co_resident_warp<TN>(P, W_comp, ctl, aux, co_warp_number(warp));
        return;
    } else {
        compute_cta<TN>(P, W_comp, ring, ctl, aux, (int)blockIdx.x - P.C);
        TL(if (threadIdx.x == 0) tl_put(P, kTlComputeEnd, globaltimer_ns()));
        // out of GEMM tiles: help with the communication that is left (all TMA and TMEM traffic is over)
        if (P.drain_help && P.mode == MOE_MODE_FUSED && !ctl->abort) comm_cta<TN>(P, W_comp, ring, ctl, aux, kRoleBack, 0);
    }
    TL(if (threadIdx.x == 0) tl_put(P, kTlCtaEnd, globaltimer_ns()));
}

// Pair kernel: launched with clusters of two CTAs.  Communication CTAs are single CTAs (blockIdx < C);
// with an odd C the cluster-mate of the last one has no role; compute pairs start at the next even index.
__global__ void __launch_bounds__(kFusedThreads, 1)
moe_gemm2_combine_pair_kernel(const __grid_constant__ FusedParams P)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // Layout: six operand stages, the control block, the aux region -- or, when nothing needs the aux region
    // while the GEMM runs (256-bit epilogue stores, no co-resident communication warp), seven stages and the
    // control block; the seventh stage then serves as the aux region of the communication role, which only
    // starts after the CTA's last MMA (drain help) or never computes (communication CTA).
    const bool seven = (P.pair_stages == 7);
    Control *ctl = reinterpret_cast<Control *>(ring + kStageBytesTotal + (seven ? PairCfg::kStageBytes : 0));
    uint8_t *aux = seven ? ring + kStageBytesTotal
                         : reinterpret_cast<uint8_t *>(ring + kStageBytesTotal + ((sizeof(Control) + 127) & ~(size_t)127));

    if (blockIdx.x == 0 && threadIdx.x < (unsigned)P.L) {
        P.split_done_next[threadIdx.x] = 0u;
        P.queue_next[threadIdx.x] = 0ull;
    }
    init_comm_barriers(ctl);
    __syncthreads();          // the only CTA-wide barrier all 20 warps share
    TL(if (threadIdx.x == 0) { tl_put(P, kTlBegin, globaltimer_ns()); tl_put(P, kTlRole, (int)blockIdx.x < ((P.C + 1) & ~1) ? 0u : 1u); });

    const int warp = threadIdx.x >> 5;
    const int c_even = (P.C + 1) & ~1;
    const int W_comp = launch_w_comp(P);
    if ((int)blockIdx.x < P.C) {
        comm_cta<256>(P, W_comp, ring, ctl, aux, P.drain_help ? kRoleFront : kRoleStatic, (int)blockIdx.x);
    } else if ((int)blockIdx.x < c_even) {
        // odd C: the last communication CTA's cluster-mate cannot compute (no partner).  With dynamic work
        // distribution it serves communication work as well; under the static map it has no tile list.
        if (P.drain_help && P.mode == MOE_MODE_FUSED) comm_cta<256>(P, W_comp, ring, ctl, aux, kRoleFront, (int)blockIdx.x);
    } else if (warp >= kThreads / 32 && P.epi_warps == 12) {
        // The compute warps of both CTAs meet at two cluster barriers (set-up and teardown), and a cluster
        // barrier counts every thread: these warps join the first, arrive at once on the second (they hold
        // nothing a peer could touch) and pick its completion up when their own work is done.
        cluster_sync_all();
        cluster_arrive();
        if (co_warp_number(warp) < P.co_warps) co_resident_warp<256>(P, W_comp, ctl, aux, co_warp_number(warp));
        cluster_wait();
        return;
    } else {
        compute_cta_pair(P, W_comp, ring, ctl, aux, ((int)blockIdx.x - c_even) >> 1);
        TL(if (threadIdx.x == 0) tl_put(P, kTlComputeEnd, globaltimer_ns()));
        if (P.drain_help && P.mode == MOE_MODE_FUSED && !ctl->abort) comm_cta<256>(P, W_comp, ring, ctl, aux, kRoleBack, 0);
    }
    TL(if (threadIdx.x == 0) tl_put(P, kTlCtaEnd, globaltimer_ns()));
}

}  // namespace

int fused_co_warps_max() { return kCoWarpsAux; }
bool fused_timeline_build() { return MOE_TIMELINE != 0; }

size_t fused_smem_bytes(int) { return (size_t)kStageBytesTotal + 1024 + ((sizeof(Control) + 127) & ~(size_t)127) + kAuxBytes; }

template <int TN>
static cudaError_t prepare()
{
    return cudaFuncSetAttribute(moe_gemm2_combine_kernel<TN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)fused_smem_bytes(TN));
}

cudaError_t fused_occupancy(int tile_n, int *blocks_per_sm)
{
    cudaError_t e;
    const size_t sm = fused_smem_bytes(tile_n);
    switch (tile_n) {
    case 64:
        if ((e = prepare<64>()) != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, moe_gemm2_combine_kernel<64>, kFusedThreads, sm);
    case 128:
        if ((e = prepare<128>()) != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, moe_gemm2_combine_kernel<128>, kFusedThreads, sm);
    case 256:
        if ((e = prepare<256>()) != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, moe_gemm2_combine_kernel<256>, kFusedThreads, sm);
    }
    return cudaErrorInvalidValue;
}

cudaError_t pair_occupancy(int *blocks_per_sm, int *max_clusters)
{
    const size_t sm = fused_smem_bytes(256);
    cudaError_t e = cudaFuncSetAttribute(moe_gemm2_combine_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, moe_gemm2_combine_pair_kernel, kFusedThreads, sm);
    if (e != cudaSuccess) return e;
    int dev = 0, n_sm = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_sm & ~1));
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = sm;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaOccupancyMaxActiveClusters(max_clusters, moe_gemm2_combine_pair_kernel, &cfg);
}

cudaError_t pair_launch(const FusedParams &p, int grid, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = fused_smem_bytes(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, moe_gemm2_combine_pair_kernel, p);
}

cudaError_t fused_launch(int tile_n, const FusedParams &p, int grid, cudaStream_t stream)
{
    const size_t sm = fused_smem_bytes(tile_n);
    switch (tile_n) {
    case 64: moe_gemm2_combine_kernel<64><<<grid, kFusedThreads, sm, stream>>>(p); break;
    case 128: moe_gemm2_combine_kernel<128><<<grid, kFusedThreads, sm, stream>>>(p); break;
    case 256: moe_gemm2_combine_kernel<256><<<grid, kFusedThreads, sm, stream>>>(p); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace moe
