// Routing / permutation / routed-tile-count builder (device).
//
// Section II-A: the router's token-expert assignments; Eq. 5: expert e needs
// ceil(M_e / T_M) tiles along the token dimension; Eq. 16: their sum S.
// The routed rows are the flat assignments f = t * k_tot + j in a *stable* order by expert.
//
// Three launch shapes, the same arithmetic and the same outputs bit for bit:
//   routing_small    up to 32 chunks of 256 assignments: one launch of one CTA;
//   routing_cluster  up to 128 chunks: one launch of one cluster of 8 CTAs, totals exchanged in
//                    distributed shared memory;
//   otherwise four small launches over the whole GPU:
//   1. hist          every warp histograms its own contiguous chunk of assignments;
//   2. scan_columns  one CTA per expert: exclusive prefix of that expert's histogram column over
//                    the warps (the per-(warp, expert) bases) and the expert's count;
//   3. finalize      one CTA: exclusive offsets, tiles per expert and their prefix, the m-tile table;
//   4. scatter       every warp walks its chunk in order, 32 assignments at a time;
//                    match_any gives each lane its rank among equal experts -> stable.

#include "moe_internal.h"

#include <cooperative_groups.h>

namespace moe {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kPerLane = kRoutingChunk / 32;   // assignments of a chunk held by one lane
static_assert(kRoutingChunk % 32 == 0, "a chunk is a whole number of warp-wide rows");

// The four launches of the large path are chained with programmatic stream serialization: a launch may be
// set up while its predecessor still runs, and waits here, first thing, until the predecessor's writes are
// visible.  Without that launch attribute this returns at once.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// launch `kernel` so that it may be set up before the previous kernel on the stream has finished
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ void report(uint32_t *status, uint32_t code, uint32_t detail, uint32_t where)
{
    if (atomicCAS(&status[0], 0u, code) == 0u) {
        status[1] = detail;
        status[2] = where;
    }
    atomicAdd(&status[3], 1u);
}

// ---- the three steps every path runs on a chunk, one warp per chunk --------------------------------------
//
// Slot i of lane l is flat assignment begin + 32 i + l.  The ids of a chunk are fetched with independent
// loads, all in flight together: a loop with one dependent load per 32 assignments spent its time on
// memory latency (8 round trips per chunk and pass).

// expert ids of the chunk (-1 past the end)
__device__ __forceinline__ void chunk_load(const int32_t *__restrict__ topk_idx, int begin, int end, int lane, int (&e)[kPerLane])
{
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        const int f = begin + 32 * i + lane;
        e[i] = f < end ? __ldg(topk_idx + f) : -1;
    }
}

// histogram of the chunk into h[E_tot] (shared memory, zeroed by the caller); bad ids and an expert chosen
// twice by one token are reported and left out / kept, as the scatter does
__device__ __forceinline__ void chunk_hist(const int32_t *__restrict__ topk_idx, int begin, int end, int lane, int k_tot,
                                           int E_tot, const int (&e)[kPerLane], int32_t *h, uint32_t *status)
{
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        const int f = begin + 32 * i + lane;
        if (f >= end) continue;
        if (e[i] < 0 || e[i] >= E_tot) {
            report(status, MOE_DEV_OOB, (uint32_t)f, 1u);
            continue;
        }
        atomicAdd(&h[e[i]], 1);
        // the same expert twice inside one token?
        const int t = f / k_tot, j = f - t * k_tot;
        for (int jj = 0; jj < j; ++jj)
            if (__ldg(topk_idx + t * k_tot + jj) == e[i]) report(status, MOE_DEV_DUP_EXPERT, (uint32_t)t, 1u);
    }
}

// stable scatter of the chunk: run[e] is the next free routed row of expert e for this chunk; match_any
// gives each lane its rank among the lanes of the row with the same expert.  off / toff: exclusive prefixes
// of the per-expert rows and m-tiles.
__device__ __forceinline__ void chunk_scatter(int begin, int end, int lane, int E_tot, int tile_m, const int (&e)[kPerLane],
                                              int32_t *run, const int32_t *off, const int32_t *toff,
                                              int32_t *__restrict__ perm, int32_t *__restrict__ inv_perm,
                                              int32_t *__restrict__ pad_row)
{
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        if (begin + 32 * i >= end) break;     // warp-uniform
        const int f = begin + 32 * i + lane;
        const bool in = f < end;
        const int ex = e[i];
        const bool ok = in && ex >= 0 && ex < E_tot;
        const unsigned active = __ballot_sync(0xffffffffu, ok);
        if (in && !ok) { inv_perm[f] = -1; pad_row[f] = -1; }
        if (ok) {
            const unsigned same = __match_any_sync(active, ex);
            const int rank = __popc(same & ((1u << lane) - 1u));
            const int r = run[ex] + rank;
            __syncwarp(active);
            if (rank == 0) run[ex] += __popc(same);
            perm[r] = f;
            inv_perm[f] = r;
            pad_row[f] = tile_m * toff[ex] + (r - off[ex]);
        }
        __syncwarp();
    }
}

// One warp: exclusive prefixes over the experts of the rows (s_off) and of the m-tiles ceil(rows / tile_m)
// (s_toff), totals in entry E_tot (Eq. 5, Eq. 16), 32 experts per step.
__device__ __forceinline__ void expert_prefix(const int32_t *s_cnt, int32_t *s_off, int32_t *s_toff, int E_tot, int tile_m, int lane)
{
    int off = 0, toff = 0;
    for (int e0 = 0; e0 < E_tot; e0 += 32) {
        const int e = e0 + lane;
        const int c = e < E_tot ? s_cnt[e] : 0;
        const int tl = (c + tile_m - 1) / tile_m;
        int ic = c, it = tl;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int uc = __shfl_up_sync(0xffffffffu, ic, d), ut = __shfl_up_sync(0xffffffffu, it, d);
            if (lane >= d) { ic += uc; it += ut; }
        }
        if (e < E_tot) {
            s_off[e] = off + ic - c;
            s_toff[e] = toff + it - tl;
        }
        off += __shfl_sync(0xffffffffu, ic, 31);
        toff += __shfl_sync(0xffffffffu, it, 31);
    }
    if (lane == 0) {
        s_off[E_tot] = off;
        s_toff[E_tot] = toff;
    }
}

// The tile counts for the host, written straight into host memory the GPU can address (`mail`, or nullptr):
// the word at mail[0] takes `seq` once tiles[0..E_tot) and S sit at mail[kMailCountsAt...].  A host that polls
// the word has the counts while the scatter still runs and needs neither a copy nor a stream synchronisation.
// Called by every thread of one CTA, after the prefixes are complete.
__device__ __forceinline__ void mail_counts(int32_t *mail, uint32_t seq, const int32_t *s_toff, int E_tot)
{
    if (!mail) return;
    for (int x = threadIdx.x; x <= E_tot; x += blockDim.x)
        mail[kMailCountsAt + x] = (x < E_tot) ? s_toff[x + 1] - s_toff[x] : s_toff[E_tot];
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence_system();
        *reinterpret_cast<volatile uint32_t *>(mail) = seq;
    }
}

// m-tile table entry mu: the expert is found by bisection in the tile prefix
__device__ __forceinline__ void mtile_entry(int mu, int E_tot, int tile_m, const int32_t *s_cnt, const int32_t *s_off,
                                            const int32_t *s_toff, int32_t *__restrict__ mtile_expert,
                                            int32_t *__restrict__ mtile_first_row, int32_t *__restrict__ mtile_valid)
{
    int lo = 0, hi = E_tot - 1;          // largest e with tile_offsets[e] <= mu
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (s_toff[mid] <= mu) lo = mid; else hi = mid - 1;
    }
    const int e = lo, i = mu - s_toff[e];
    mtile_expert[mu] = e;
    mtile_first_row[mu] = s_off[e] + i * tile_m;
    mtile_valid[mu] = min(tile_m, s_cnt[e] - i * tile_m);
}

// ---- large batches: four launches over the whole GPU -------------------------------------------------------

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
routing_hist(const int32_t *__restrict__ topk_idx, int R, int k_tot, int E_tot, int n_warps,
             int32_t *__restrict__ whist, uint32_t *status)
{
    extern __shared__ int32_t sh[];
    const int warp_in_block = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int w = blockIdx.x * kWarpsPerBlock + warp_in_block;
    if (w >= n_warps) return;
    int32_t *h = sh + warp_in_block * E_tot;
    const int begin = w * kRoutingChunk, end = min(R, begin + kRoutingChunk);
    int e[kPerLane];
    chunk_load(topk_idx, begin, end, lane, e);
    for (int x = lane; x < E_tot; x += 32) h[x] = 0;
    __syncwarp();
    chunk_hist(topk_idx, begin, end, lane, k_tot, E_tot, e, h, status);
    __syncwarp();
    for (int x = lane; x < E_tot; x += 32) whist[(size_t)w * E_tot + x] = h[x];
}

// Per expert (one CTA each): counts[e], and whist[.][e] turned into an exclusive prefix over the
// sorting warps.  Thread t owns a contiguous run of warps; the run sums are scanned across the CTA.
constexpr int kScanThreads = 256;
__global__ void __launch_bounds__(kScanThreads)
routing_scan_columns(int E_tot, int n_warps, int32_t *__restrict__ whist, int32_t *__restrict__ counts)
{
    __shared__ int warp_sum[kScanThreads / 32];
    grid_dependency_wait();
    const int e = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int chunk = (n_warps + kScanThreads - 1) / kScanThreads;
    const int w_lo = min(n_warps, tid * chunk), w_hi = min(n_warps, w_lo + chunk);
    int sum = 0;
    for (int w = w_lo; w < w_hi; ++w) sum += whist[(size_t)w * E_tot + e];
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    if (lane == 31) warp_sum[wid] = incl;
    __syncthreads();
    int base = incl - sum;
    for (int i = 0; i < wid; ++i) base += warp_sum[i];
    for (int w = w_lo; w < w_hi; ++w) {
        const int c = whist[(size_t)w * E_tot + e];
        whist[(size_t)w * E_tot + e] = base;
        base += c;
    }
    if (tid == kScanThreads - 1) counts[e] = base;
}

// Offsets, tile counts and the m-tile table from the per-expert counts (one CTA).
// Dynamic shared memory: 3 * (E_tot + 1) ints.
__global__ void __launch_bounds__(1024)
routing_finalize(int E_tot, int tile_m, int max_mtiles, const int32_t *__restrict__ counts,
                 int32_t *__restrict__ offsets, int32_t *__restrict__ tiles, int32_t *__restrict__ tile_offsets,
                 int32_t *__restrict__ mtile_expert, int32_t *__restrict__ mtile_first_row,
                 int32_t *__restrict__ mtile_valid, uint32_t *status, int32_t *mail, uint32_t mail_seq)
{
    extern __shared__ int32_t fin[];
    grid_dependency_wait();
    int32_t *s_cnt = fin, *s_off = fin + (E_tot + 1), *s_toff = fin + 2 * (E_tot + 1);
    for (int e = threadIdx.x; e < E_tot; e += blockDim.x) s_cnt[e] = counts[e];
    __syncthreads();
    if (threadIdx.x < 32) expert_prefix(s_cnt, s_off, s_toff, E_tot, tile_m, threadIdx.x);
    __syncthreads();
    mail_counts(mail, mail_seq, s_toff, E_tot);
    if (threadIdx.x == 0 && s_toff[E_tot] > max_mtiles) report(status, MOE_DEV_OOB, (uint32_t)s_toff[E_tot], 2u);
    for (int e = threadIdx.x; e <= E_tot; e += blockDim.x) {
        offsets[e] = s_off[e];
        tile_offsets[e] = s_toff[e];
        // S rides behind the per-expert tile counts for the host copy
        tiles[e] = (e < E_tot) ? s_toff[e + 1] - s_toff[e] : s_toff[E_tot];
    }
    const int S = min(s_toff[E_tot], max_mtiles);
    for (int mu = threadIdx.x; mu < S; mu += blockDim.x)
        mtile_entry(mu, E_tot, tile_m, s_cnt, s_off, s_toff, mtile_expert, mtile_first_row, mtile_valid);
}

// Dynamic shared memory: (kWarpsPerBlock * E_tot + 2 * (E_tot + 1)) ints.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
routing_scatter(const int32_t *__restrict__ topk_idx, int R, int E_tot, int tile_m, int n_warps,
                const int32_t *__restrict__ whist, const int32_t *__restrict__ offsets,
                const int32_t *__restrict__ tile_offsets, int32_t *__restrict__ perm,
                int32_t *__restrict__ inv_perm, int32_t *__restrict__ pad_row)
{
    extern __shared__ int32_t sh[];
    const int warp_in_block = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int w = blockIdx.x * kWarpsPerBlock + warp_in_block;
    const int begin = min(R, w * kRoutingChunk), end = w < n_warps ? min(R, begin + kRoutingChunk) : begin;
    // the ids do not depend on the launches before this one: fetch them before waiting
    int e[kPerLane];
    chunk_load(topk_idx, begin, end, lane, e);
    grid_dependency_wait();
    int32_t *s_off = sh + kWarpsPerBlock * E_tot, *s_toff = s_off + (E_tot + 1);
    for (int x = threadIdx.x; x <= E_tot; x += blockDim.x) {
        s_off[x] = offsets[x];
        s_toff[x] = tile_offsets[x];
    }
    __syncthreads();
    if (w >= n_warps) return;
    int32_t *run = sh + warp_in_block * E_tot;  // next free row per expert, for this warp
    for (int x = lane; x < E_tot; x += 32) run[x] = s_off[x] + whist[(size_t)w * E_tot + x];
    __syncwarp();
    chunk_scatter(begin, end, lane, E_tot, tile_m, e, run, s_off, s_toff, perm, inv_perm, pad_row);
}

// ---- small batches: the same steps in ONE launch of one CTA ------------------------------------------------
//
// At most 32 chunks (8192 assignments), one per warp; the per-chunk histograms live in shared memory, the ids
// of a chunk stay in its warp's registers from the histogram to the scatter, the steps are separated by CTA
// barriers instead of launch boundaries.  Same arithmetic, same outputs, bit for bit; four launches cost
// ~30 us of which the work is a few microseconds at these sizes.
constexpr int kSmallWarps = 32;
constexpr size_t kSmallMaxSmem = 200 * 1024;
__global__ void __launch_bounds__(kSmallWarps * 32)
routing_small(const int32_t *__restrict__ topk_idx, int R, int k_tot, int E_tot, int tile_m, int n_chunks, int max_mtiles,
              int32_t *__restrict__ counts, int32_t *__restrict__ offsets, int32_t *__restrict__ tiles,
              int32_t *__restrict__ tile_offsets, int32_t *__restrict__ mtile_expert,
              int32_t *__restrict__ mtile_first_row, int32_t *__restrict__ mtile_valid, int32_t *__restrict__ perm,
              int32_t *__restrict__ inv_perm, int32_t *__restrict__ pad_row, uint32_t *status, int32_t *mail,
              uint32_t mail_seq)
{
    extern __shared__ int32_t sm[];
    int32_t *whist = sm;                                   // [kSmallWarps][E_tot]
    int32_t *s_cnt = sm + kSmallWarps * E_tot, *s_off = s_cnt + (E_tot + 1), *s_toff = s_off + (E_tot + 1);
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t *h = whist + w * E_tot;
    const int begin = min(R, w * kRoutingChunk), end = w < n_chunks ? min(R, begin + kRoutingChunk) : begin;
    // 1. histogram of the warp's chunk
    int e[kPerLane];
    chunk_load(topk_idx, begin, end, lane, e);
    for (int x = lane; x < E_tot; x += 32) h[x] = 0;
    __syncwarp();
    chunk_hist(topk_idx, begin, end, lane, k_tot, E_tot, e, h, status);
    __syncthreads();
    // 2. per expert: exclusive prefix of its histogram column over the chunks, and its count
    for (int x = threadIdx.x; x < E_tot; x += blockDim.x) {
        int base = 0;
        for (int c = 0; c < n_chunks; ++c) {
            const int v = whist[c * E_tot + x];
            whist[c * E_tot + x] = base;
            base += v;
        }
        s_cnt[x] = base;
        counts[x] = base;
    }
    __syncthreads();
    // 3. offsets, tiles per expert and their prefix, the m-tile table
    if (w == 0) expert_prefix(s_cnt, s_off, s_toff, E_tot, tile_m, lane);
    __syncthreads();
    mail_counts(mail, mail_seq, s_toff, E_tot);
    if (threadIdx.x == 0 && s_toff[E_tot] > max_mtiles) report(status, MOE_DEV_OOB, (uint32_t)s_toff[E_tot], 2u);
    for (int x = threadIdx.x; x <= E_tot; x += blockDim.x) {
        offsets[x] = s_off[x];
        tile_offsets[x] = s_toff[x];
        tiles[x] = (x < E_tot) ? s_toff[x + 1] - s_toff[x] : s_toff[E_tot];
    }
    const int S = min(s_toff[E_tot], max_mtiles);
    for (int mu = threadIdx.x; mu < S; mu += blockDim.x)
        mtile_entry(mu, E_tot, tile_m, s_cnt, s_off, s_toff, mtile_expert, mtile_first_row, mtile_valid);
    // 4. stable scatter of the warp's chunk: h[x] becomes the next free row of expert x for this chunk
    for (int x = lane; x < E_tot; x += 32) h[x] += s_off[x];
    __syncwarp();
    chunk_scatter(begin, end, lane, E_tot, tile_m, e, h, s_off, s_toff, perm, inv_perm, pad_row);
}

// ---- medium batches: ONE launch of one thread-block cluster ------------------------------------------------
//
// CTA r of the cluster owns a contiguous run of chunks, one per warp, and keeps their histograms in its own
// shared memory; the per-expert totals of the CTAs are exchanged through distributed shared memory (the only
// step that crosses CTAs), the launch boundaries become one cluster barrier.  Same outputs as the other two
// paths, bit for bit.  Measured on B200 against the four launches: 8 CTAs win ~10 us at 128 chunks and
// lose ~12 us at 512; a single CTA is 2x slower than four launches at 128 chunks.
constexpr int kClusterCtas = 8;
constexpr int kClusterMaxChunks = 128;
static_assert(kClusterMaxChunks <= kClusterCtas * kSmallWarps, "one chunk per warp");
__global__ void __launch_bounds__(kSmallWarps * 32)
routing_cluster(const int32_t *__restrict__ topk_idx, int R, int k_tot, int E_tot, int tile_m, int n_chunks, int max_mtiles,
                int32_t *__restrict__ counts, int32_t *__restrict__ offsets, int32_t *__restrict__ tiles,
                int32_t *__restrict__ tile_offsets, int32_t *__restrict__ mtile_expert,
                int32_t *__restrict__ mtile_first_row, int32_t *__restrict__ mtile_valid, int32_t *__restrict__ perm,
                int32_t *__restrict__ inv_perm, int32_t *__restrict__ pad_row, uint32_t *status, int32_t *mail,
                uint32_t mail_seq)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int nb = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int cpc = (n_chunks + nb - 1) / nb;                       // chunks per CTA (<= 32), a contiguous run
    const int c_lo = min(n_chunks, rank * cpc), c_n = min(n_chunks, c_lo + cpc) - c_lo;
    extern __shared__ int32_t sm[];
    int32_t *whist = sm;                                            // [cpc][E_tot]
    int32_t *s_tot = sm + (size_t)cpc * E_tot;                      // this CTA's rows per expert (read by the others)
    int32_t *s_base = s_tot + E_tot;                                // rows per expert in the CTAs before this one
    int32_t *s_cnt = s_base + E_tot, *s_off = s_cnt + (E_tot + 1), *s_toff = s_off + (E_tot + 1);
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool mine = w < c_n;                                      // this warp has a chunk
    int32_t *h = whist + (size_t)(mine ? w : 0) * E_tot;
    const int begin = min(R, (c_lo + w) * kRoutingChunk), end = mine ? min(R, begin + kRoutingChunk) : begin;
    // 1. histogram of the warp's chunk
    int e[kPerLane];
    chunk_load(topk_idx, begin, end, lane, e);
    if (mine) {
        for (int x = lane; x < E_tot; x += 32) h[x] = 0;
        __syncwarp();
        chunk_hist(topk_idx, begin, end, lane, k_tot, E_tot, e, h, status);
    }
    __syncthreads();
    // 2. per expert: exclusive prefix over this CTA's chunks, the CTA's total; then the totals of all CTAs
    for (int x = threadIdx.x; x < E_tot; x += blockDim.x) {
        int base = 0;
        for (int lc = 0; lc < c_n; ++lc) {
            const int v = whist[(size_t)lc * E_tot + x];
            whist[(size_t)lc * E_tot + x] = base;
            base += v;
        }
        s_tot[x] = base;
    }
    cluster.sync();
    for (int x = threadIdx.x; x < E_tot; x += blockDim.x) {
        int before = 0, total = 0;
        for (int j = 0; j < nb; ++j) {
            const int v = cluster.map_shared_rank(s_tot, j)[x];
            if (j < rank) before += v;
            total += v;
        }
        s_base[x] = before;
        s_cnt[x] = total;
        if (rank == 0) counts[x] = total;
    }
    __syncthreads();
    // 3. offsets, tiles per expert and their prefix (every CTA, for its own scatter), the m-tile table
    if (w == 0) expert_prefix(s_cnt, s_off, s_toff, E_tot, tile_m, lane);
    __syncthreads();
    if (rank == 0) {
        mail_counts(mail, mail_seq, s_toff, E_tot);
        if (threadIdx.x == 0 && s_toff[E_tot] > max_mtiles) report(status, MOE_DEV_OOB, (uint32_t)s_toff[E_tot], 2u);
        for (int x = threadIdx.x; x <= E_tot; x += blockDim.x) {
            offsets[x] = s_off[x];
            tile_offsets[x] = s_toff[x];
            tiles[x] = (x < E_tot) ? s_toff[x + 1] - s_toff[x] : s_toff[E_tot];
        }
    }
    const int S = min(s_toff[E_tot], max_mtiles);
    for (int mu = rank * blockDim.x + threadIdx.x; mu < S; mu += nb * blockDim.x)
        mtile_entry(mu, E_tot, tile_m, s_cnt, s_off, s_toff, mtile_expert, mtile_first_row, mtile_valid);
    // 4. stable scatter of the warp's chunk: h[x] becomes the next free row of expert x for this chunk
    if (mine) {
        for (int x = lane; x < E_tot; x += 32) h[x] += s_off[x] + s_base[x];
        __syncwarp();
        chunk_scatter(begin, end, lane, E_tot, tile_m, e, h, s_off, s_toff, perm, inv_perm, pad_row);
    }
    cluster.sync();   // no CTA leaves while another may still read its totals
}

size_t routing_cluster_smem(int n_chunks, int E_tot)
{
    const int cpc = (n_chunks + kClusterCtas - 1) / kClusterCtas;
    return ((size_t)cpc * E_tot + 2 * (size_t)E_tot + 3 * (size_t)(E_tot + 1)) * sizeof(int32_t);
}

cudaError_t routing_cluster_launch(const int32_t *topk_idx, const moe_shape &s, int tile_m, int R, int n_chunks,
                                   const moe_routing &r, uint32_t *status, int32_t *mail, uint32_t mail_seq, cudaStream_t stream)
{
    const size_t sm = routing_cluster_smem(n_chunks, s.E_tot);
    if (sm > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(routing_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmallMaxSmem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kClusterCtas);
    cfg.blockDim = dim3(kSmallWarps * 32);
    cfg.dynamicSmemBytes = sm;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kClusterCtas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, routing_cluster, topk_idx, R, (int)s.k_tot, (int)s.E_tot, tile_m, n_chunks,
                              (int)r.max_mtiles, r.counts, r.offsets, r.tiles, r.tile_offsets, r.mtile_expert,
                              r.mtile_first_row, r.mtile_valid, r.perm, r.inv_perm, r.pad_row, status, mail, mail_seq);
}

// the four launches; `scratch`: n_chunks * E_tot ints that need not start at any value
cudaError_t routing_four_launches(const int32_t *topk_idx, const moe_shape &s, int tile_m, int R, int n_chunks,
                                  const moe_routing &r, int32_t *scratch, uint32_t *status, int32_t *mail, uint32_t mail_seq,
                                  cudaStream_t stream)
{
    const int blocks = (n_chunks + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int E = (int)s.E_tot;
    const size_t sh_hist = (size_t)kWarpsPerBlock * E * sizeof(int32_t);
    const size_t sh_scat = sh_hist + 2 * (size_t)(E + 1) * sizeof(int32_t);
    if (blocks > 0)
        routing_hist<<<blocks, kWarpsPerBlock * 32, sh_hist, stream>>>(topk_idx, R, s.k_tot, E, n_chunks, scratch, status);
    cudaError_t e = launch_chained(routing_scan_columns, dim3(E), dim3(kScanThreads), 0, stream, E, n_chunks, scratch, r.counts);
    if (e != cudaSuccess) return e;
    e = launch_chained(routing_finalize, dim3(1), dim3(1024), 3 * (size_t)(E + 1) * sizeof(int32_t), stream, E, tile_m,
                       (int)r.max_mtiles, r.counts, r.offsets, r.tiles, r.tile_offsets, r.mtile_expert, r.mtile_first_row,
                       r.mtile_valid, status, mail, mail_seq);
    if (e != cudaSuccess) return e;
    if (blocks > 0)
        e = launch_chained(routing_scatter, dim3(blocks), dim3(kWarpsPerBlock * 32), sh_scat, stream, topk_idx, R, E, tile_m,
                           n_chunks, scratch, r.offsets, r.tile_offsets, r.perm, r.inv_perm, r.pad_row);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace

cudaError_t routing_launch(const int32_t *topk_idx, const moe_shape &s, int tile_m, const moe_routing &r, uint32_t *status,
                           int32_t *mail, uint32_t mail_seq, cudaStream_t stream)
{
    const int R = s.T * s.k_tot;
    const int n_chunks = (R + kRoutingChunk - 1) / kRoutingChunk;
    const size_t sm_small = ((size_t)kSmallWarps * s.E_tot + 3 * (size_t)(s.E_tot + 1)) * sizeof(int32_t);
    if (n_chunks <= kSmallWarps && sm_small <= kSmallMaxSmem) {
        if (sm_small > 48 * 1024) {
            const cudaError_t e = cudaFuncSetAttribute(routing_small, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmallMaxSmem);
            if (e != cudaSuccess) return e;
        }
        routing_small<<<1, kSmallWarps * 32, sm_small, stream>>>(
            topk_idx, R, s.k_tot, s.E_tot, tile_m, n_chunks, r.max_mtiles, r.counts, r.offsets, r.tiles, r.tile_offsets,
            r.mtile_expert, r.mtile_first_row, r.mtile_valid, r.perm, r.inv_perm, r.pad_row, status, mail, mail_seq);
        return cudaGetLastError();
    }
    if (n_chunks <= kClusterMaxChunks && routing_cluster_smem(n_chunks, s.E_tot) <= kSmallMaxSmem)
        return routing_cluster_launch(topk_idx, s, tile_m, R, n_chunks, r, status, mail, mail_seq, stream);
    return routing_four_launches(topk_idx, s, tile_m, R, n_chunks, r, r.scratch, status, mail, mail_seq, stream);
}

}  // namespace moe

// ------------------------------------------------------------------------------------------
// Routing build for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving loop whose
// memory pool was sized and frozen at start-up, under a framework allocator that forbids
// foreign allocations once a model is loaded, or in a latency-critical section where an
// allocation (an implicit device synchronisation) is not acceptable.  For them the per-warp
// histograms that the builder needs as scratch live in a fixed array inside the library instead
// of in a caller-provided buffer.  Every GPU that loads the library holds the array
// (kStaticScratchInts * 4 bytes) until the process exits.
//
// `g_static_scratch` is a device symbol: in host code the name is only a host-side stand-in, not
// a device address, so the address the kernels get comes from cudaGetSymbolAddress(), looked up
// once per device with that device current.
namespace moe {
namespace {

constexpr int kStaticScratchInts = 128 * 1024;   // 512 KiB per GPU
constexpr int kMaxStaticDevices = 64;

static __device__ __align__(256) int32_t g_static_scratch[kStaticScratchInts];
int32_t *g_static_scratch_addr[kMaxStaticDevices] = {nullptr};

}  // namespace
}  // namespace moe

extern "C" int32_t moe_build_routing_static(moe_handle *h, const int32_t *topk_idx, const moe_shape *s,
                                            int32_t tile_m, const moe_routing *r,
                                            int32_t *tile_counts_host, uint32_t *status_dev, void *stream)
{
    using namespace moe;
    if (!h || !s || !r || !status_dev) return MOE_ERR_NULL;
    if (s->T < 0 || s->k_tot < 1 || s->k_tot > 32 || s->E_tot < 1 || s->E_tot > 1024 ||
        (int64_t)s->T * s->k_tot >= (int64_t)1 << 30)
        return MOE_ERR_SHAPE;
    if (tile_m != 64 && tile_m != 128 && tile_m != 256) return MOE_ERR_UNSUPPORTED;
    if (s->T > 0 && !topk_idx) return MOE_ERR_NULL;
    const int64_t R = (int64_t)s->T * s->k_tot;
    if (r->max_mtiles < (int32_t)(R / tile_m + s->E_tot)) return MOE_ERR_SHAPE;
    const int64_t n_warps = (R + kRoutingChunk - 1) / kRoutingChunk;
    if (n_warps * s->E_tot > kStaticScratchInts) {
        snprintf(h->err, sizeof h->err,
                 "moe_build_routing_static: ceil(T*k_tot/%d) * E_tot = %lld ints of scratch needed, the built-in "
                 "array holds %d; use moe_build_routing with a caller-allocated workspace",
                 kRoutingChunk, (long long)(n_warps * s->E_tot), kStaticScratchInts);
        return MOE_ERR_STATIC_LIMIT;
    }
    if (h->device < 0 || h->device >= kMaxStaticDevices) return MOE_ERR_UNSUPPORTED;
    // Every call, not only the first: the kernels below run on the CURRENT device, and the array's
    // address is only meaningful on the device it was resolved for.  A caller whose current device
    // is not the handle's gets an error instead of kernels that dereference another GPU's address.
    {
        const int32_t rc = require_handle_device(h, "moe_build_routing_static");
        if (rc != MOE_OK) return rc;
    }

    // set-up, once per device: resolve the array's device address (the handle's device is current)
    int32_t *scratch = g_static_scratch_addr[h->device];
    if (!scratch) {
        void *p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) return cuda_fail(h, e, "cudaGetSymbolAddress(static scratch)");
        scratch = static_cast<int32_t *>(p);
        g_static_scratch_addr[h->device] = scratch;   // every writer stores the same value
    }

    // The array keeps whatever the previous call left in it.  Nothing has to start at zero: the
    // histogram pass overwrites every (warp, expert) entry the later passes read.
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = routing_four_launches(topk_idx, *s, tile_m, (int)R, (int)n_warps, *r, scratch, status_dev, nullptr, 0u, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "static routing launch");
    if (tile_counts_host) {
        e = cudaMemcpyAsync(tile_counts_host, r->tiles, (size_t)(s->E_tot + 1) * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(h, e, "tile counts copy");
    }
    return MOE_OK;
}
