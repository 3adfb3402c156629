// Internal declarations shared by the translation units of libmoe_b200.so.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <unordered_map>

#include "../../include/moe_b200.h"

namespace moe {

constexpr int kThreads = 512;          // threads of a CTA's compute (or dedicated communication) role: 16 warps
constexpr int kCoWarpsMax = 4;         // co-resident communication warps a compute CTA of the fused kernel may carry
constexpr int kFusedThreads = kThreads + 32 * kCoWarpsMax;   // block size of the fused kernel
constexpr int kBlockK = 64;            // bf16 elements per k-block: one 128-byte swizzle row
constexpr int kUmmaK = 16;             // K of one tcgen05.mma.kind::f16 instruction
constexpr int kMmaM = 128;             // M of the MMA (tile_m = 64 stores the first 64 rows only)
constexpr int kStageBytesTotal = 192 * 1024;  // operand ring, all stages together
constexpr int kCommTileM = 128;        // T_M^comm
constexpr int kCommTileN = 1024;       // T_N^comm
constexpr int kMailCountsAt = 32;      // the handle's count mailbox: word 0 = sequence number, counts from here on
constexpr int kMailInts = kMailCountsAt + 1024 + 1 + 31;
constexpr int kRoutingChunk = 256;     // flat assignments handled by one warp while sorting
constexpr uint64_t kDefaultWaitNs = 2000000000ull;
constexpr int kTimelineSlots = 40;     // 64-bit words per CTA in a timeline buffer (timeline build only)

// Parameters of one fused launch.  Passed by value (__grid_constant__): the two tensor maps
// must sit in kernel parameter space, 64-byte aligned.
struct alignas(64) FusedParams {
    CUtensorMap tmA;   // x_routed [R, I]      box 64 x 128 rows, 128B swizzle
    CUtensorMap tmB;   // W2 [E_tot, H, I]     box 64 x tile_n x 1, 128B swizzle
    const int32_t *mtile_expert;
    const int32_t *mtile_first_row;
    const int32_t *mtile_valid;
    const int32_t *S_dev;          // != nullptr: the m-tile count is read here by the kernel (S and W_comp below are unset)
    const int32_t *pad_row;
    const int32_t *perm;
    const float *topk_w;
    void *Y;                       // bf16 [T][L][slabs][Q][slab cols], token-major
    uint32_t *flags;               // [L * W_comp] readiness per global tile (== epoch when ready)
    uint32_t *split_done;          // [L] tiles finished per split (this launch)
    uint32_t *split_done_next;     // [L] counters of the next launch, zeroed by this one
    unsigned long long *queue;     // [L] drain help: items of the split handed out so far, front | back << 32
    unsigned long long *queue_next;  // [L] ... of the next launch, zeroed by this one
    uint32_t *status;              // 4 words
    unsigned long long *timeline;  // timeline build: per-CTA records, then one stamp per split; else nullptr
    uint32_t probe;                // timeline build: parts of the data movement left out (moe_set_probe); else 0
    void *out[MOE_MAX_EP];
    unsigned long long wait_ns;
    long long R_pad;
    int32_t T, H, K, TP, EP, L, k_tot;
    int32_t S, tile_m, NTs, split_w, W_comp;
    int32_t C, P, mode, withhold;
    int32_t tok_blk, tok_tiles_per_rank, comm_cols, comm_tiles;
    int32_t num_kb, last_ksteps;
    int32_t drain_help;                 // compute CTAs serve communication tiles once their GEMM tiles are done
    int32_t co_warps;                   // co-resident communication warps per compute CTA (0..2)
    int32_t pair_stages;                // operand stages of the CTA-pair kernel: 6, or 7 when the aux region of shared memory is
                                        // free during the GEMM (256-bit epilogue stores, no co-resident warp)
    int32_t epi_warps;                  // epilogue warps of a compute CTA: 12 (warps 4-15), or 16 (warps 4-19) when no
                                        // co-resident warp is asked for and the epilogue needs no staging buffer
    int32_t tile_order;                 // 0: split-major tile sequence (the paper's); 1: m-tile-major across splits
    int32_t flag_parts;                 // readiness flags per tile: 1, or 2 for a CTA-pair tile
    int32_t Q, slab_cols, slab_shift;   // Q = k_tot * TP rows per unit; slab_cols = 1 << slab_shift
    int32_t wide_store;                 // every 16-column group of a Y row is whole and 32-byte aligned: 256-bit epilogue stores
    uint32_t epoch;
};

}  // namespace moe

namespace moe {
// what the two operand tensor maps of the fused kernel depend on
struct TensorMapKey {
    const void *x, *w2;
    int32_t T, k_tot, I, H, E_tot, box_n;
};
}  // namespace moe

struct moe_handle {
    int device = 0;
    int G = 0;
    unsigned long long wait_ns = moe::kDefaultWaitNs;
    char err[512] = {0};
    std::unordered_map<const void *, uint32_t> epochs;  // per flags workspace
    void *encode_tiled = nullptr;                       // cuTensorMapEncodeTiled
    int o_comp[3] = {0, 0, 0};                          // tile_n = 64, 128, 256
    int o_pair = 0;                                     // CTA-pair kernel: resident CTAs per SM
    int max_pairs = 0;                                  // ... and co-resident clusters of two
    // Mailbox for the routed-tile counts (Section III-E: the manager reads them on the host): pinned host
    // memory the GPU writes directly.  The routing kernel stores tiles[0..E_tot) and S at
    // mail[kMailCountsAt...] and then the call's sequence number at mail[0]; the whole-step calls poll that
    // word instead of queueing a copy and synchronising the stream.
    int32_t *mail_host = nullptr;
    int32_t *mail_dev = nullptr;                        // the same memory as the GPU addresses it
    uint32_t mail_seq = 0;
    void *counts_event = nullptr;                       // cudaEvent_t: "the tile counts have reached the host"
    unsigned long long *timeline = nullptr;             // timeline build: where the next fused launch records
    size_t timeline_bytes = 0;
    uint32_t probe = 0;                                 // timeline build: moe_set_probe bits for the next launches
    CUtensorMap tmA, tmB;                               // last encoded operand tensor maps of the fused kernel ...
    moe::TensorMapKey tm_key = {};                      // ... and what they were encoded for
    bool tm_valid = false;
};

namespace moe {

inline int tile_n_slot(int tile_n) { return tile_n == 64 ? 0 : tile_n == 128 ? 1 : tile_n == 256 ? 2 : -1; }

int32_t cuda_fail(moe_handle *h, cudaError_t e, const char *what);
// MOE_OK when the calling thread's current CUDA device is the handle's; MOE_ERR_UNSUPPORTED (with a
// message in the handle) otherwise.  Every launching entry point checks it: kernels run on the
// current device, the buffers and the cached residency belong to the handle's.
int32_t require_handle_device(moe_handle *h, const char *who);
// fused kernel (gemm2_combine.cu)
size_t fused_smem_bytes(int tile_n);
cudaError_t fused_occupancy(int tile_n, int *blocks_per_sm);
cudaError_t fused_launch(int tile_n, const FusedParams &p, int grid, cudaStream_t stream);
int fused_co_warps_max();
bool fused_timeline_build();   // the library was compiled with -DMOE_TIMELINE=1   // co-resident communication warps a compute CTA has shared memory for
// CTA-pair kernel (256 x 256 tiles, clusters of two)
cudaError_t pair_occupancy(int *blocks_per_sm, int *max_clusters);
cudaError_t pair_launch(const FusedParams &p, int grid, cudaStream_t stream);
// routing kernels (routing.cu)
// mail / mail_seq: see moe_handle::mail_host (nullptr: the counts are not mailed)
cudaError_t routing_launch(const int32_t *topk_idx, const moe_shape &s, int tile_m, const moe_routing &r, uint32_t *status,
                           int32_t *mail, uint32_t mail_seq, cudaStream_t stream);

}  // namespace moe
