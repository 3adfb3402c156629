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

__device__ __forceinline__ void report(uint32_t *status, uint32_t code, uint32_t detail, uint32_t where)
{
    if (atomicCAS(&status[0], 0u, code) == 0u) {
        status[1] = detail;
        status[2] = where;
    }
    atomicAdd(&status[3], 1u);
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
routing_hist(const int32_t *__restrict__ topk_idx, int R, int k_tot, int E_tot, int n_warps,
             int32_t *__restrict__ whist, uint32_t *status)
{
    extern __shared__ int32_t sh[];
    const int warp_in_block = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int w = blockIdx.x * kWarpsPerBlock + warp_in_block;
    int32_t *h = sh + warp_in_block * E_tot;
    for (int e = lane; e < E_tot; e += 32) h[e] = 0;
    __syncwarp();
    if (w < n_warps) {
        const int begin = w * kRoutingChunk;
        const int end = min(R, begin + kRoutingChunk);
        for (int f = begin + lane; f < end; f += 32) {
            const int e = topk_idx[f];
            if (e < 0 || e >= E_tot) {
                report(status, MOE_DEV_OOB, (uint32_t)f, 1u);
                continue;
            }
            atomicAdd(&h[e], 1);
            // the same expert twice inside one token?
            const int t = f / k_tot, j = f - t * k_tot;
            for (int jj = 0; jj < j; ++jj)
                if (topk_idx[t * k_tot + jj] == e) report(status, MOE_DEV_DUP_EXPERT, (uint32_t)t, 1u);
        }
        __syncwarp();
        for (int e = lane; e < E_tot; e += 32) whist[(size_t)w * E_tot + e] = h[e];
    }
}

// Per expert (one CTA each): counts[e], and whist[.][e] turned into an exclusive prefix over the
// sorting warps.  Thread t owns a contiguous run of warps; the run sums are scanned across the CTA.
constexpr int kScanThreads = 256;
__global__ void __launch_bounds__(kScanThreads)
routing_scan_columns(int E_tot, int n_warps, int32_t *__restrict__ whist, int32_t *__restrict__ counts)
{
    __shared__ int warp_sum[kScanThreads / 32];
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

// Offsets, tile counts and the m-tile table from the per-expert counts (one CTA; the prefix over the
// experts is serial but runs in shared memory).  Dynamic shared memory: 3 * (E_tot + 1) ints.
__global__ void __launch_bounds__(1024)
routing_finalize(int E_tot, int tile_m, int max_mtiles, const int32_t *__restrict__ counts,
                 int32_t *__restrict__ offsets, int32_t *__restrict__ tiles, int32_t *__restrict__ tile_offsets,
                 int32_t *__restrict__ mtile_expert, int32_t *__restrict__ mtile_first_row,
                 int32_t *__restrict__ mtile_valid, uint32_t *status)
{
    extern __shared__ int32_t fin[];
    int32_t *s_cnt = fin, *s_off = fin + (E_tot + 1), *s_toff = fin + 2 * (E_tot + 1);
    for (int e = threadIdx.x; e < E_tot; e += blockDim.x) s_cnt[e] = counts[e];
    __syncthreads();
    if (threadIdx.x == 0) {
        int off = 0, toff = 0;
        for (int e = 0; e < E_tot; ++e) {
            s_off[e] = off;
            s_toff[e] = toff;
            off += s_cnt[e];
            toff += (s_cnt[e] + tile_m - 1) / tile_m;
        }
        s_off[E_tot] = off;
        s_toff[E_tot] = toff;
        if (toff > max_mtiles) report(status, MOE_DEV_OOB, (uint32_t)toff, 2u);
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E_tot; e += blockDim.x) {
        offsets[e] = s_off[e];
        tile_offsets[e] = s_toff[e];
        // S rides behind the per-expert tile counts for the host copy
        tiles[e] = (e < E_tot) ? s_toff[e + 1] - s_toff[e] : s_toff[E_tot];
    }
    // m-tile table, one thread per m-tile: the expert is found by bisection in the tile prefix
    const int S = min(s_toff[E_tot], max_mtiles);
    for (int mu = threadIdx.x; mu < S; mu += blockDim.x) {
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
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
routing_scatter(const int32_t *__restrict__ topk_idx, int R, int E_tot, int tile_m, int n_warps,
                const int32_t *__restrict__ whist, const int32_t *__restrict__ offsets,
                const int32_t *__restrict__ tile_offsets, int32_t *__restrict__ perm,
                int32_t *__restrict__ inv_perm, int32_t *__restrict__ pad_row)
{
    extern __shared__ int32_t sh[];
    const int warp_in_block = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int w = blockIdx.x * kWarpsPerBlock + warp_in_block;
    if (w >= n_warps) return;
    int32_t *run = sh + warp_in_block * E_tot;  // next free row per expert, for this warp
    for (int e = lane; e < E_tot; e += 32) run[e] = offsets[e] + whist[(size_t)w * E_tot + e];
    __syncwarp();
    const int begin = w * kRoutingChunk;
    const int end = min(R, begin + kRoutingChunk);
    for (int f0 = begin; f0 < end; f0 += 32) {
        const int f = f0 + lane;
        const bool in = f < end;
        int e = in ? topk_idx[f] : -1;
        const bool ok = in && e >= 0 && e < E_tot;
        const unsigned active = __ballot_sync(0xffffffffu, ok);
        if (in && !ok) { inv_perm[f] = -1; pad_row[f] = -1; }
        if (ok) {
            const unsigned same = __match_any_sync(active, e);
            const int rank = __popc(same & ((1u << lane) - 1u));
            const int r = run[e] + rank;
            __syncwarp(active);
            if (rank == 0) run[e] += __popc(same);
            perm[r] = f;
            inv_perm[f] = r;
            pad_row[f] = tile_m * tile_offsets[e] + (r - offsets[e]);
        }
        __syncwarp();
    }
}

// The same four steps in ONE launch of one CTA, for small and decode-sized batches (at most 32 chunks of
// 256 assignments, at most 256 experts): the per-warp histograms live in shared memory, the steps are
// separated by CTA barriers instead of launch boundaries.  Same arithmetic, same outputs, bit for bit; four
// launches cost ~30 us of which the work is a few microseconds at these sizes.
constexpr int kSmallWarps = 32;
constexpr int kSmallMaxExperts = 256;
__global__ void __launch_bounds__(kSmallWarps * 32)
routing_small(const int32_t *__restrict__ topk_idx, int R, int k_tot, int E_tot, int tile_m, int n_warps, int max_mtiles,
              int32_t *__restrict__ counts, int32_t *__restrict__ offsets, int32_t *__restrict__ tiles,
              int32_t *__restrict__ tile_offsets, int32_t *__restrict__ mtile_expert,
              int32_t *__restrict__ mtile_first_row, int32_t *__restrict__ mtile_valid, int32_t *__restrict__ perm,
              int32_t *__restrict__ inv_perm, int32_t *__restrict__ pad_row, uint32_t *status)
{
    extern __shared__ int32_t sm[];
    int32_t *whist = sm;                                   // [kSmallWarps][E_tot]
    int32_t *s_cnt = sm + kSmallWarps * E_tot, *s_off = s_cnt + (E_tot + 1), *s_toff = s_off + (E_tot + 1);
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t *h = whist + w * E_tot;
    // 1. per-warp histograms of the warp's chunk
    for (int e = lane; e < E_tot; e += 32) h[e] = 0;
    __syncwarp();
    const int begin = w * kRoutingChunk;
    const int end = w < n_warps ? min(R, begin + kRoutingChunk) : begin;
    for (int f = begin + lane; f < end; f += 32) {
        const int e = topk_idx[f];
        if (e < 0 || e >= E_tot) {
            report(status, MOE_DEV_OOB, (uint32_t)f, 1u);
            continue;
        }
        atomicAdd(&h[e], 1);
        const int t = f / k_tot, j = f - t * k_tot;
        for (int jj = 0; jj < j; ++jj)
            if (topk_idx[t * k_tot + jj] == e) report(status, MOE_DEV_DUP_EXPERT, (uint32_t)t, 1u);
    }
    __syncthreads();
    // 2. per expert: exclusive prefix of its histogram column over the warps, and its count
    for (int e = threadIdx.x; e < E_tot; e += blockDim.x) {
        int base = 0;
        for (int ww = 0; ww < n_warps; ++ww) {
            const int c = whist[ww * E_tot + e];
            whist[ww * E_tot + e] = base;
            base += c;
        }
        s_cnt[e] = base;
        counts[e] = base;
    }
    __syncthreads();
    // 3. offsets, tiles per expert and their prefix, the m-tile table
    if (threadIdx.x == 0) {
        int off = 0, toff = 0;
        for (int e = 0; e < E_tot; ++e) {
            s_off[e] = off;
            s_toff[e] = toff;
            off += s_cnt[e];
            toff += (s_cnt[e] + tile_m - 1) / tile_m;
        }
        s_off[E_tot] = off;
        s_toff[E_tot] = toff;
        if (toff > max_mtiles) report(status, MOE_DEV_OOB, (uint32_t)toff, 2u);
    }
    __syncthreads();
    for (int e = threadIdx.x; e <= E_tot; e += blockDim.x) {
        offsets[e] = s_off[e];
        tile_offsets[e] = s_toff[e];
        tiles[e] = (e < E_tot) ? s_toff[e + 1] - s_toff[e] : s_toff[E_tot];
    }
    const int S = min(s_toff[E_tot], max_mtiles);
    for (int mu = threadIdx.x; mu < S; mu += blockDim.x) {
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
    // 4. stable scatter of the warp's chunk: h[e] becomes the next free row of expert e for this warp
    for (int e = lane; e < E_tot; e += 32) h[e] += s_off[e];
    __syncwarp();
    for (int f0 = begin; f0 < end; f0 += 32) {
        const int f = f0 + lane;
        const bool in = f < end;
        int e = in ? topk_idx[f] : -1;
        const bool ok = in && e >= 0 && e < E_tot;
        const unsigned active = __ballot_sync(0xffffffffu, ok);
        if (in && !ok) { inv_perm[f] = -1; pad_row[f] = -1; }
        if (ok) {
            const unsigned same = __match_any_sync(active, e);
            const int rank = __popc(same & ((1u << lane) - 1u));
            const int r = h[e] + rank;
            __syncwarp(active);
            if (rank == 0) h[e] += __popc(same);
            perm[r] = f;
            inv_perm[f] = r;
            pad_row[f] = tile_m * s_toff[e] + (r - s_off[e]);
        }
        __syncwarp();
    }
}

// The four steps in ONE launch of one thread-block cluster, for the batches between the single-CTA kernel
// and the sizes where the whole GPU pays: CTA r of the cluster owns a contiguous run of chunks and keeps
// their histograms in its own shared memory; the per-expert totals of the CTAs are exchanged through
// distributed shared memory (the only step that crosses CTAs), the launch boundaries become one cluster
// barrier.  Same arithmetic and outputs as the other two paths, bit for bit.
// Measured on B200: against the four launches, 8 CTAs win ~10 us at 128 chunks and lose ~12 us at 512.
constexpr int kClusterCtas = 8;
constexpr int kClusterMaxChunks = 128;
constexpr size_t kClusterMaxSmem = 200 * 1024;
__global__ void __launch_bounds__(kSmallWarps * 32)
routing_cluster(const int32_t *__restrict__ topk_idx, int R, int k_tot, int E_tot, int tile_m, int n_chunks, int max_mtiles,
                int32_t *__restrict__ counts, int32_t *__restrict__ offsets, int32_t *__restrict__ tiles,
                int32_t *__restrict__ tile_offsets, int32_t *__restrict__ mtile_expert,
                int32_t *__restrict__ mtile_first_row, int32_t *__restrict__ mtile_valid, int32_t *__restrict__ perm,
                int32_t *__restrict__ inv_perm, int32_t *__restrict__ pad_row, uint32_t *status)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int nb = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int cpc = (n_chunks + nb - 1) / nb;                       // chunks per CTA, a contiguous run
    const int c_lo = min(n_chunks, rank * cpc), c_n = min(n_chunks, c_lo + cpc) - c_lo;
    extern __shared__ int32_t sm[];
    int32_t *whist = sm;                                            // [cpc][E_tot]
    int32_t *s_tot = sm + (size_t)cpc * E_tot;                      // this CTA's rows per expert (read by the others)
    int32_t *s_base = s_tot + E_tot;                                // rows per expert in the CTAs before this one
    int32_t *s_cnt = s_base + E_tot, *s_off = s_cnt + (E_tot + 1), *s_toff = s_off + (E_tot + 1);
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // 1. histogram of every chunk of this CTA (by the warp that will scatter it)
    for (int lc = w; lc < c_n; lc += kSmallWarps) {
        int32_t *h = whist + (size_t)lc * E_tot;
        for (int e = lane; e < E_tot; e += 32) h[e] = 0;
        __syncwarp();
        const int begin = (c_lo + lc) * kRoutingChunk, end = min(R, begin + kRoutingChunk);
        for (int f = begin + lane; f < end; f += 32) {
            const int e = topk_idx[f];
            if (e < 0 || e >= E_tot) {
                report(status, MOE_DEV_OOB, (uint32_t)f, 1u);
                continue;
            }
            atomicAdd(&h[e], 1);
            const int t = f / k_tot, j = f - t * k_tot;
            for (int jj = 0; jj < j; ++jj)
                if (topk_idx[t * k_tot + jj] == e) report(status, MOE_DEV_DUP_EXPERT, (uint32_t)t, 1u);
        }
    }
    __syncthreads();
    // 2. per expert: exclusive prefix over this CTA's chunks, and the CTA's total
    for (int e = threadIdx.x; e < E_tot; e += blockDim.x) {
        int base = 0;
        for (int lc = 0; lc < c_n; ++lc) {
            const int v = whist[(size_t)lc * E_tot + e];
            whist[(size_t)lc * E_tot + e] = base;
            base += v;
        }
        s_tot[e] = base;
    }
    cluster.sync();
    for (int e = threadIdx.x; e < E_tot; e += blockDim.x) {
        int before = 0, total = 0;
        for (int j = 0; j < nb; ++j) {
            const int v = cluster.map_shared_rank(s_tot, j)[e];
            if (j < rank) before += v;
            total += v;
        }
        s_base[e] = before;
        s_cnt[e] = total;
        if (rank == 0) counts[e] = total;
    }
    __syncthreads();
    // 3. offsets, tiles per expert and their prefix (every CTA, for its own scatter), the m-tile table
    if (threadIdx.x == 0) {
        int off = 0, toff = 0;
        for (int e = 0; e < E_tot; ++e) {
            s_off[e] = off;
            s_toff[e] = toff;
            off += s_cnt[e];
            toff += (s_cnt[e] + tile_m - 1) / tile_m;
        }
        s_off[E_tot] = off;
        s_toff[E_tot] = toff;
        if (rank == 0 && toff > max_mtiles) report(status, MOE_DEV_OOB, (uint32_t)toff, 2u);
    }
    __syncthreads();
    if (rank == 0)
        for (int e = threadIdx.x; e <= E_tot; e += blockDim.x) {
            offsets[e] = s_off[e];
            tile_offsets[e] = s_toff[e];
            tiles[e] = (e < E_tot) ? s_toff[e + 1] - s_toff[e] : s_toff[E_tot];
        }
    const int S = min(s_toff[E_tot], max_mtiles);
    for (int mu = rank * blockDim.x + threadIdx.x; mu < S; mu += nb * blockDim.x) {
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
    // 4. stable scatter, chunk by chunk: h[e] becomes the next free row of expert e for this chunk
    for (int lc = w; lc < c_n; lc += kSmallWarps) {
        int32_t *h = whist + (size_t)lc * E_tot;
        for (int e = lane; e < E_tot; e += 32) h[e] += s_off[e] + s_base[e];
        __syncwarp();
        const int begin = (c_lo + lc) * kRoutingChunk, end = min(R, begin + kRoutingChunk);
        for (int f0 = begin; f0 < end; f0 += 32) {
            const int f = f0 + lane;
            const bool in = f < end;
            int e = in ? topk_idx[f] : -1;
            const bool ok = in && e >= 0 && e < E_tot;
            const unsigned active = __ballot_sync(0xffffffffu, ok);
            if (in && !ok) { inv_perm[f] = -1; pad_row[f] = -1; }
            if (ok) {
                const unsigned same = __match_any_sync(active, e);
                const int rk = __popc(same & ((1u << lane) - 1u));
                const int r = h[e] + rk;
                __syncwarp(active);
                if (rk == 0) h[e] += __popc(same);
                perm[r] = f;
                inv_perm[f] = r;
                pad_row[f] = tile_m * s_toff[e] + (r - s_off[e]);
            }
            __syncwarp();
        }
    }
    cluster.sync();   // no CTA leaves while another may still read its totals
}

size_t routing_cluster_smem(int n_chunks, int E_tot)
{
    const int cpc = (n_chunks + kClusterCtas - 1) / kClusterCtas;
    return ((size_t)cpc * E_tot + 2 * (size_t)E_tot + 3 * (size_t)(E_tot + 1)) * sizeof(int32_t);
}

cudaError_t routing_cluster_launch(const int32_t *topk_idx, const moe_shape &s, int tile_m, int R, int n_chunks,
                                   const moe_routing &r, uint32_t *status, cudaStream_t stream)
{
    const size_t sm = routing_cluster_smem(n_chunks, s.E_tot);
    cudaError_t e = cudaSuccess;
    if (sm > 48 * 1024)
        e = cudaFuncSetAttribute(routing_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kClusterMaxSmem);
    if (e != cudaSuccess) return e;
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
                              r.mtile_first_row, r.mtile_valid, r.perm, r.inv_perm, r.pad_row, status);
}

}  // namespace

cudaError_t routing_launch(const int32_t *topk_idx, const moe_shape &s, int tile_m,
                           const moe_routing &r, uint32_t *status, cudaStream_t stream)
{
    const int R = s.T * s.k_tot;
    const int n_warps = (R + kRoutingChunk - 1) / kRoutingChunk;
    if (n_warps <= kSmallWarps && s.E_tot <= kSmallMaxExperts) {
        const size_t sm = ((size_t)kSmallWarps * s.E_tot + 3 * (size_t)(s.E_tot + 1)) * sizeof(int32_t);
        routing_small<<<1, kSmallWarps * 32, sm, stream>>>(
            topk_idx, R, s.k_tot, s.E_tot, tile_m, n_warps, r.max_mtiles, r.counts, r.offsets, r.tiles, r.tile_offsets,
            r.mtile_expert, r.mtile_first_row, r.mtile_valid, r.perm, r.inv_perm, r.pad_row, status);
        return cudaGetLastError();
    }
    if (n_warps <= kClusterMaxChunks && routing_cluster_smem(n_warps, s.E_tot) <= kClusterMaxSmem)
        return routing_cluster_launch(topk_idx, s, tile_m, R, n_warps, r, status, stream);
    const int blocks = (n_warps + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const size_t sh = (size_t)kWarpsPerBlock * s.E_tot * sizeof(int32_t);
    if (blocks > 0)
        routing_hist<<<blocks, kWarpsPerBlock * 32, sh, stream>>>(topk_idx, R, s.k_tot, s.E_tot, n_warps,
                                                                  r.scratch, status);
    routing_scan_columns<<<s.E_tot, kScanThreads, 0, stream>>>(s.E_tot, n_warps, r.scratch, r.counts);
    routing_finalize<<<1, 1024, 3 * (size_t)(s.E_tot + 1) * sizeof(int32_t), stream>>>(
        s.E_tot, tile_m, r.max_mtiles, r.counts, r.offsets, r.tiles, r.tile_offsets, r.mtile_expert,
        r.mtile_first_row, r.mtile_valid, status);
    if (blocks > 0)
        routing_scatter<<<blocks, kWarpsPerBlock * 32, sh, stream>>>(
            topk_idx, R, s.E_tot, tile_m, n_warps, r.scratch, r.offsets, r.tile_offsets, r.perm,
            r.inv_perm, r.pad_row);
    return cudaGetLastError();
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
    const int iR = (int)R, nw = (int)n_warps;
    const int blocks = (nw + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const size_t sh = (size_t)kWarpsPerBlock * s->E_tot * sizeof(int32_t);
    if (blocks > 0)
        routing_hist<<<blocks, kWarpsPerBlock * 32, sh, st>>>(topk_idx, iR, s->k_tot, s->E_tot, nw, scratch, status_dev);
    routing_scan_columns<<<s->E_tot, kScanThreads, 0, st>>>(s->E_tot, nw, scratch, r->counts);
    routing_finalize<<<1, 1024, 3 * (size_t)(s->E_tot + 1) * sizeof(int32_t), st>>>(
        s->E_tot, tile_m, r->max_mtiles, r->counts, r->offsets, r->tiles, r->tile_offsets, r->mtile_expert,
        r->mtile_first_row, r->mtile_valid, status_dev);
    if (blocks > 0)
        routing_scatter<<<blocks, kWarpsPerBlock * 32, sh, st>>>(topk_idx, iR, s->E_tot, tile_m, nw, scratch,
                                                                r->offsets, r->tile_offsets, r->perm,
                                                                r->inv_perm, r->pad_row);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e, "static routing launch");
    if (tile_counts_host) {
        e = cudaMemcpyAsync(tile_counts_host, r->tiles, (size_t)(s->E_tot + 1) * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(h, e, "tile counts copy");
    }
    return MOE_OK;
}
