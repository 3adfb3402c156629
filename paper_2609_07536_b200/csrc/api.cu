// Host side of the C ABI: handle, workspace layout, argument validation, tensor maps, launches.

#include <climits>
#include <cstdint>
#include <cstring>
#include <new>

#include <algorithm>

#include "moe_internal.h"

#include <atomic>
#include <chrono>

namespace moe {

int32_t cuda_fail(moe_handle *h, cudaError_t e, const char *what)
{
    if (h) snprintf(h->err, sizeof h->err, "%s: %s", what, cudaGetErrorString(e));
    return MOE_ERR_CUDA;
}

int32_t require_handle_device(moe_handle *h, const char *who)
{
    int cur = -1;
    const cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return cuda_fail(h, e, "cudaGetDevice");
    if (cur != h->device) {
        snprintf(h->err, sizeof h->err, "%s: the current CUDA device is %d, the handle was created on device %d",
                 who, cur, h->device);
        return MOE_ERR_UNSUPPORTED;
    }
    return MOE_OK;
}

namespace {

inline size_t align16(size_t x) { return (x + 15) & ~(size_t)15; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

constexpr int64_t kPairTileMinRowsPerExpert = 192;   // mean routed rows per expert from which 256-row pair tiles pay
constexpr int kSplitCounterWords = 64;  // 2 parities x MOE_MAX_L split counters (32-bit), then 2 x MOE_MAX_L work queues (64-bit), padded

bool shape_ok(const moe_shape *s)
{
    return s->T >= 0 && s->H >= 8 && s->I >= 16 && s->E_tot >= 1 && s->E_tot <= 1024 && s->k_tot >= 1 &&
           s->k_tot <= 32 && s->TP >= 1 && s->TP <= 8 && s->EP >= 1 && s->EP <= MOE_MAX_EP && s->L >= 1 &&
           s->L <= MOE_MAX_L && s->H % 8 == 0 && s->I % s->TP == 0 && (s->I / s->TP) % 16 == 0 &&
           (int64_t)s->T * s->k_tot < (int64_t)1 << 30;
}
bool tile_ok(int tile_m, int tile_n)
{
    return ((tile_m == 64 || tile_m == 128) && tile_n_slot(tile_n) >= 0) || (tile_m == 256 && tile_n == 256);
}
bool tile_m_ok(int tile_m) { return tile_m == 64 || tile_m == 128 || tile_m == 256; }

int32_t max_mtiles_of(const moe_shape *s, int tile_m)
{
    return (int32_t)((int64_t)s->T * s->k_tot / tile_m + s->E_tot);
}
int32_t n_routing_warps(const moe_shape *s)
{
    return (int32_t)ceil_div((int64_t)s->T * s->k_tot, kRoutingChunk);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

}  // namespace
}  // namespace moe

using namespace moe;

#ifndef MOE_PAIR_SEVENTH_STAGE
#define MOE_PAIR_SEVENTH_STAGE 1
#endif
static constexpr bool kPairSeventhStage = MOE_PAIR_SEVENTH_STAGE != 0;

extern "C" {

int32_t moe_create(int32_t device, moe_handle **out)
{
    if (!out) return MOE_ERR_NULL;
    *out = nullptr;
    moe_handle *h = new (std::nothrow) moe_handle();
    if (!h) return MOE_ERR_CUDA;
    h->device = device;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->G, cudaDevAttrMultiProcessorCount, device);
    int major = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e != cudaSuccess || major != 10) {
        delete h;
        return e != cudaSuccess ? MOE_ERR_CUDA : MOE_ERR_UNSUPPORTED;
    }
    cudaDriverEntryPointQueryResult q;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &h->encode_tiled, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !h->encode_tiled) {
        delete h;
        return MOE_ERR_CUDA;
    }
    const int tns[3] = {64, 128, 256};
    for (int i = 0; i < 3; ++i) {
        e = fused_occupancy(tns[i], &h->o_comp[i]);
        if (e != cudaSuccess) {
            delete h;
            return MOE_ERR_CUDA;
        }
    }
    e = pair_occupancy(&h->o_pair, &h->max_pairs);
    if (e != cudaSuccess) {
        delete h;
        return MOE_ERR_CUDA;
    }
    cudaEvent_t ev = nullptr;
    e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        delete h;
        return MOE_ERR_CUDA;
    }
    h->counts_event = ev;
    // the count mailbox: a few KB of pinned host memory that the GPU addresses directly.  Without it (the
    // allocation or the mapping refused) the whole-step calls copy the counts and synchronise instead.
    void *mail = nullptr, *mail_dev = nullptr;
    if (cudaHostAlloc(&mail, (size_t)kMailInts * sizeof(int32_t), cudaHostAllocMapped | cudaHostAllocPortable) == cudaSuccess) {
        memset(mail, 0, (size_t)kMailInts * sizeof(int32_t));
        if (cudaHostGetDevicePointer(&mail_dev, mail, 0) == cudaSuccess && mail_dev) {
            h->mail_host = static_cast<int32_t *>(mail);
            h->mail_dev = static_cast<int32_t *>(mail_dev);
        } else {
            cudaFreeHost(mail);
        }
    }
    (void)cudaGetLastError();
    *out = h;
    return MOE_OK;
}

int32_t moe_destroy(moe_handle *h)
{
    if (h && h->counts_event) cudaEventDestroy(static_cast<cudaEvent_t>(h->counts_event));
    if (h && h->mail_host) cudaFreeHost(h->mail_host);
    delete h;
    return MOE_OK;
}

const char *moe_last_cuda_error(const moe_handle *h) { return h ? h->err : ""; }

int32_t moe_set_wait_limit_ns(moe_handle *h, uint64_t ns)
{
    if (!h) return MOE_ERR_NULL;
    h->wait_ns = ns;
    return MOE_OK;
}

int32_t moe_set_timeline(moe_handle *h, void *timeline_dev, size_t bytes)
{
    if (!h) return MOE_ERR_NULL;
    if (timeline_dev && !fused_timeline_build()) {
        snprintf(h->err, sizeof h->err, "moe_set_timeline: this library was built without -DMOE_TIMELINE=1");
        return MOE_ERR_UNSUPPORTED;
    }
    if (timeline_dev && (reinterpret_cast<uintptr_t>(timeline_dev) & 7u)) return MOE_ERR_ALIGN;
    h->timeline = static_cast<unsigned long long *>(timeline_dev);
    h->timeline_bytes = timeline_dev ? bytes : 0;
    return MOE_OK;
}

int32_t moe_set_probe(moe_handle *h, uint32_t probe_bits)
{
    if (!h) return MOE_ERR_NULL;
    if (probe_bits && !fused_timeline_build()) {
        snprintf(h->err, sizeof h->err, "moe_set_probe: this library was built without -DMOE_TIMELINE=1");
        return MOE_ERR_UNSUPPORTED;
    }
    if (probe_bits & ~63u) return MOE_ERR_SHAPE;
    h->probe = probe_bits;
    return MOE_OK;
}

int32_t moe_query_occupancy(moe_handle *h, int32_t tile_m, int32_t tile_n, moe_occupancy *occ,
                            moe_sm_limits *limits, moe_rho *rho)
{
    if (!h) return MOE_ERR_NULL;
    if (!tile_ok(tile_m, tile_n)) return MOE_ERR_UNSUPPORTED;
    if (occ) {
        occ->tile_m = tile_m;
        occ->tile_n = tile_n;
        occ->comm_tile_m = kCommTileM;
        occ->comm_tile_n = kCommTileN;
        // both roles are CTAs of the same kernel: one resident CTA per SM by shared memory
        const bool pair = (tile_m == 256);
        occ->o_comp = pair ? h->o_pair : h->o_comp[tile_n_slot(tile_n)];
        occ->o_comm = occ->o_comp;
        occ->comp_slot_sms = pair ? 2 : 1;
    }
    if (limits) {
        // a pair tile needs both CTAs of a cluster resident: count only SMs that can host one
        limits->G = (tile_m == 256) ? (2 * h->max_pairs < h->G ? 2 * h->max_pairs : h->G) : h->G;
        limits->C_max = h->G / 2;   // one-time saturation characterisation of this kernel family
        limits->force_comm_ctas = 0;
        limits->selector_off = 0;
        limits->default_C = 3;      // the fixed count of the upstream path (Section II-C)
        limits->drain_help = 1;
        limits->co_warps_max = fused_co_warps_max();
        limits->force_co_warps = -1;
        limits->C_co_max = 8;       // beside co-resident warps more dedicated CTAs than this never paid (one-time sweep)
        limits->dep_model = MOE_DEP_SPLIT;
        // Lower end of the co-resident family's legal set (one-time sweep).  One-CTA tiles: below 24 compute waves
        // co-resident warps lost 2-5 % (T = 1024: 19 waves; T = 2048: 37).  CTA-pair tiles: a co-resident warp takes
        // the shared memory of the seventh operand stage, and with seven stages for w = 0 the best w > 0 candidate
        // never beat the best w = 0 one at any size of the sweep (1.00-1.05 of it): the family is not offered (a
        // forced w is still honoured).
        limits->co_min_waves = (tile_m == 256) ? INT32_MAX : 24;
    }
    if (rho) {
        // One-time service-rate characterisation of this kernel family on B200 (Eq. 13), one constant per
        // GEMM tile shape (Section III-E: every kernel choice brings its own).  Reference run: DeepSeek-V2-
        // Lite shape, T = 4096, uniform routing, TP = 2, EP = 2, L = 2, K = 704; each role alone on its
        // share of the SMs at C = 32: time per communication wave / time per compute wave.
        //   128x256: 70.8 us / 5.88 us ; 256x256 (CTA pair): 71.0 / 4.75 ; 128x128: 70.6 / 3.97
        rho->K_ref = 704;
        rho->tile_m_ref = tile_m;
        rho->tile_n_ref = tile_n;
        if (tile_m == 256) rho->rho_ref = 14.96;
        else if (tile_n == 256) rho->rho_ref = 12.04;
        else if (tile_n == 128) rho->rho_ref = 17.80;
        else rho->rho_ref = 17.80 * 2.0;          // 64-wide tiles: Eq. 14 tile-area scaling from 128x128
        if (tile_m == 64) rho->rho_ref *= 1.0;     // a 64-row tile still occupies a 128-row MMA: same wave time
        if (tile_n == 64) { rho->tile_n_ref = 64; }
        rho->D_ref = 2;
        rho->rows_ref = 8 * 2 + 1;
        rho->comm_cols_ref = 1024;
        rho->mode = MOE_RHO_LOCAL;
        // Warp-level capacity and bandwidth coupling, measured once on B200 (DeepSeek-V2-Lite shape):
        //   a communication CTA is 12 warps; alone it streams 68 GB/s (5.7 GB/s per warp), 148 of them together
        //   5.85 TB/s (the copy bandwidth): 5850 / 5.67 = 1030 warps saturate HBM;
        //   a co-resident warp beside a running GEMM serves 2.6-2.8 GB/s (2.2 times slower than a dedicated warp)
        //   and each one stretches the compute wave by 1.25 % (683 -> 704 -> 714 us of GEMM phase for w = 0, 1, 2,
        //   of which 2 % is the split-major tile order that w > 0 needs when L > 1: x is read once per split).
        //   the dynamic hand-out gives out single tokens of a communication tile (T_M^comm pieces per tile).
        rho->comm_warps_per_cta = 12;
        rho->comm_quanta_per_tile = kCommTileM;
        rho->reserved0 = 0;
        rho->n_sat_warps = 1030;
        rho->co_beta = 0.0125;
        rho->co_gamma = 2.2;
        rho->co_order = 0.02;
    }
    return MOE_OK;
}

int32_t moe_select_tile(moe_handle *h, const moe_shape *s, int32_t *tile_m, int32_t *tile_n)
{
    if (!h || !s || !tile_m || !tile_n) return MOE_ERR_NULL;
    if (!shape_ok(s)) return MOE_ERR_SHAPE;
    // Conventional kernel dispatch (Section III-E: it runs before the resource manager and hands it the tile
    // shape and residency of the kernel it chose).  Widest n-tile the split holds; rows: the 256-row CTA-pair
    // tile moves a third less operand traffic per FLOP but pads every expert's last tile to 256 rows and needs
    // two co-scheduled SMs, so it pays once an expert fills most of one such tile on average (measured on the
    // DeepSeek-V2-Lite shape, fused kernel, 128x256 against 256x256: 78 / 100 us at T = 16, 128 / 132 at 1024
    // (124 rows per expert), 172 / 160 at 2048 (248 rows), 257 / 243 at 4096, 466 / 423 at 8192, 885 / 791 at
    // 16384; Qwen shape (546 rows per expert) 265 / 242, Granite shape (819 rows, K = 256) 134 / 131).
    const int64_t split_w = ceil_div(s->H, s->L);
    const int32_t tn = split_w >= 256 ? 256 : split_w >= 128 ? 128 : 64;
    const int64_t rows_per_expert = (int64_t)s->T * s->k_tot / s->E_tot;
    const bool pair = tn == 256 && h->max_pairs > 0 && rows_per_expert >= kPairTileMinRowsPerExpert;
    *tile_m = pair ? 256 : 128;
    *tile_n = tn;
    return MOE_OK;
}

int32_t moe_workspace_bytes(const moe_shape *s, int32_t tile_m, int32_t tile_n, size_t *routing_bytes,
                            size_t *y_bytes, size_t *flags_bytes, size_t *status_bytes)
{
    if (!s) return MOE_ERR_NULL;
    if (!shape_ok(s)) return MOE_ERR_SHAPE;
    if (!tile_ok(tile_m, tile_n)) return MOE_ERR_UNSUPPORTED;
    const size_t R = (size_t)s->T * s->k_tot, E = (size_t)s->E_tot;
    const size_t mt = (size_t)max_mtiles_of(s, tile_m);
    if (routing_bytes) {
        size_t b = 0;
        b += align16(E * 4) + 3 * align16((E + 1) * 4);  // counts, offsets, tiles(+S), tile_offsets
        b += 3 * align16(R * 4);                          // perm, inv_perm, pad_row
        b += 3 * align16(mt * 4);                         // m-tile table
        b += align16((size_t)n_routing_warps(s) * E * 4); // per-warp histograms
        *routing_bytes = b + 16;
    }
    if (y_bytes)   // token-major: [T][L][k_tot * TP][ceil(H/L)]
        *y_bytes = align16((size_t)s->T * s->L * s->k_tot * s->TP * (size_t)ceil_div(s->H, s->L) * 2) + 16;
    if (flags_bytes) {
        const size_t nts = (size_t)ceil_div(ceil_div(s->H, s->L), tile_n);
        const size_t parts = (tile_m == 256) ? 2 : 1;   // a pair tile is published in two parts
        *flags_bytes = ((size_t)kSplitCounterWords + (size_t)s->L * s->TP * mt * nts * parts) * 4 + 16;
    }
    if (status_bytes) *status_bytes = 16;
    return MOE_OK;
}

int32_t moe_routing_view(void *ws, const moe_shape *s, int32_t tile_m, moe_routing *out)
{
    if (!ws || !s || !out) return MOE_ERR_NULL;
    if (!shape_ok(s)) return MOE_ERR_SHAPE;
    if (!tile_m_ok(tile_m)) return MOE_ERR_UNSUPPORTED;
    if (!aligned16(ws)) return MOE_ERR_ALIGN;
    const size_t R = (size_t)s->T * s->k_tot, E = (size_t)s->E_tot;
    const size_t mt = (size_t)max_mtiles_of(s, tile_m);
    char *p = static_cast<char *>(ws);
    auto take = [&](size_t n_ints) {
        int32_t *q = reinterpret_cast<int32_t *>(p);
        p += align16(n_ints * 4);
        return q;
    };
    out->counts = take(E);
    out->offsets = take(E + 1);
    out->tiles = take(E + 1);
    out->tile_offsets = take(E + 1);
    out->perm = take(R);
    out->inv_perm = take(R);
    out->pad_row = take(R);
    out->mtile_expert = take(mt);
    out->mtile_first_row = take(mt);
    out->mtile_valid = take(mt);
    out->scratch = take((size_t)n_routing_warps(s) * E);
    out->max_mtiles = (int32_t)mt;
    return MOE_OK;
}

int32_t moe_build_routing(moe_handle *h, const int32_t *topk_idx, const moe_shape *s, int32_t tile_m,
                          const moe_routing *r, int32_t *tile_counts_host, uint32_t *status_dev, void *stream)
{
    if (!h || !s || !r || !status_dev) return MOE_ERR_NULL;
    if (!shape_ok(s)) return MOE_ERR_SHAPE;
    if (!tile_m_ok(tile_m)) return MOE_ERR_UNSUPPORTED;
    if (s->T > 0 && !topk_idx) return MOE_ERR_NULL;
    if (r->max_mtiles < max_mtiles_of(s, tile_m)) return MOE_ERR_SHAPE;
    if (const int32_t rc = require_handle_device(h, "moe_build_routing")) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = routing_launch(topk_idx, *s, tile_m, *r, status_dev, nullptr, 0u, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "routing launch");
    if (tile_counts_host) {
        e = cudaMemcpyAsync(tile_counts_host, r->tiles, (size_t)(s->E_tot + 1) * 4, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(h, e, "tile counts copy");
    }
    return MOE_OK;
}

}  // extern "C"

namespace {

// Routing build of the whole-step calls.  With the handle's mailbox the kernel that finishes the counts stores
// them into host memory itself and `*seq` is the number to wait for (wait_counts); without it, the plain
// build with its copy, and `*seq` = 0.
int32_t build_routing_mailed(moe_handle *h, const int32_t *topk_idx, const moe_shape *s, int32_t tile_m, const moe_routing *r,
                             int32_t *tile_counts_host, uint32_t *status_dev, cudaStream_t st, uint32_t *seq)
{
    *seq = 0;
    if (!tile_counts_host || !h->mail_dev)
        return moe_build_routing(h, topk_idx, s, tile_m, r, tile_counts_host, status_dev, st);
    if (!s || !r || !status_dev) return MOE_ERR_NULL;
    if (!shape_ok(s)) return MOE_ERR_SHAPE;
    if (!tile_m_ok(tile_m)) return MOE_ERR_UNSUPPORTED;
    if (s->T > 0 && !topk_idx) return MOE_ERR_NULL;
    if (r->max_mtiles < max_mtiles_of(s, tile_m)) return MOE_ERR_SHAPE;
    if (const int32_t rc = require_handle_device(h, "moe_build_routing")) return rc;
    if (++h->mail_seq == 0u) h->mail_seq = 1u;
    const cudaError_t e = routing_launch(topk_idx, *s, tile_m, *r, status_dev, h->mail_dev, h->mail_seq, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "routing launch");
    *seq = h->mail_seq;
    return MOE_OK;
}

// Waits until the counts of build `seq` are on the host and copies them to tile_counts_host (E_tot + 1 ints).
// seq = 0: they come by the stream's copy: `fallback_event` if given (recorded behind that copy), else the stream.
int32_t wait_counts(moe_handle *h, uint32_t seq, int32_t E_tot, int32_t *tile_counts_host, cudaStream_t st, cudaEvent_t fallback_event)
{
    if (seq == 0u) {
        const cudaError_t e = fallback_event ? cudaEventSynchronize(fallback_event) : cudaStreamSynchronize(st);
        return e == cudaSuccess ? MOE_OK : cuda_fail(h, e, "tile counts wait");
    }
    volatile uint32_t *word = reinterpret_cast<volatile uint32_t *>(h->mail_host);
    const auto t0 = std::chrono::steady_clock::now();
    uint32_t spins = 0;
    while (*word != seq) {
        if ((++spins & 2047u) == 0u) {
            // the kernels finished or failed without the word arriving?
            const cudaError_t q = cudaStreamQuery(st);
            if (q != cudaErrorNotReady) {
                if (*word == seq) break;
                if (q != cudaSuccess) return cuda_fail(h, q, "routing build");
                snprintf(h->err, sizeof h->err, "the routing build finished without delivering the tile counts");
                return MOE_ERR_CUDA;
            }
            const double waited = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
            if (waited > 2.0 + 2e-9 * (double)h->wait_ns) {
                snprintf(h->err, sizeof h->err, "no tile counts from the routing build after %.1f s", waited);
                return MOE_ERR_CUDA;
            }
        }
#if defined(__x86_64__) || defined(__i386__)
        __builtin_ia32_pause();
#endif
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    memcpy(tile_counts_host, h->mail_host + kMailCountsAt, (size_t)(E_tot + 1) * sizeof(int32_t));
    return MOE_OK;
}

}  // namespace

extern "C" {

int32_t moe_gemm2_combine(moe_handle *h, const void *x_routed, const void *W2, const int32_t *topk_idx,
                          const float *topk_w, const moe_shape *s, const moe_occupancy *occ,
                          const moe_routing *r, int32_t n_mtiles, const moe_plan *plan, void *const *out,
                          void *y_ws, uint32_t *flags_ws, uint32_t *status_dev, void *stream)
{
    (void)topk_idx;
    if (!h || !s || !occ || !r || !plan || !out || !status_dev) return MOE_ERR_NULL;
    if (!shape_ok(s)) return MOE_ERR_SHAPE;
    if (!tile_ok(occ->tile_m, occ->tile_n)) return MOE_ERR_UNSUPPORTED;
    if (occ->comm_tile_m != kCommTileM || occ->comm_tile_n != kCommTileN) return MOE_ERR_UNSUPPORTED;
    if ((ceil_div(s->H, s->L) % 8) != 0) return MOE_ERR_SHAPE;   // 16-byte column chunks per split
    if (s->T == 0) return MOE_OK;
    if (!x_routed || !W2 || !topk_w || !y_ws || !flags_ws) return MOE_ERR_NULL;
    const bool counts_on_device = (n_mtiles == MOE_MTILES_ON_DEVICE);
    if (counts_on_device) n_mtiles = r->max_mtiles;   // bound for the sizes checked on the host
    if (n_mtiles < 0 || n_mtiles > r->max_mtiles) return MOE_ERR_SHAPE;
    if (!aligned16(x_routed) || !aligned16(W2) || !aligned16(y_ws) || !aligned16(flags_ws) ||
        !aligned16(status_dev))
        return MOE_ERR_ALIGN;
    for (int d = 0; d < s->EP; ++d) {
        if (!out[d]) return MOE_ERR_NULL;
        if (!aligned16(out[d])) return MOE_ERR_ALIGN;
    }
    const int mode = plan->mode;
    if (mode != MOE_MODE_FUSED && mode != MOE_MODE_GEMM_ONLY && mode != MOE_MODE_COMBINE_ONLY)
        return MOE_ERR_SHAPE;
    const int C = (mode == MOE_MODE_GEMM_ONLY) ? 0 : plan->comm_ctas;
    const int Pc = (mode == MOE_MODE_COMBINE_ONLY) ? 0 : plan->P;
    const int o_comp = occ->o_comp > 0 ? occ->o_comp : 1, o_comm = occ->o_comm > 0 ? occ->o_comm : 1;
    const bool pair = (occ->tile_m == 256);
    const int slot_sms = pair ? 2 : 1;
    if (occ->comp_slot_sms != slot_sms) return MOE_ERR_UNSUPPORTED;
    // without a communication CTA somebody else has to serve the communication work: the compute CTAs, once
    // their GEMM tiles are done (drain help)
    if (mode != MOE_MODE_GEMM_ONLY && (C < 0 || (C < 1 && !(mode == MOE_MODE_FUSED && plan->drain_help))))
        return MOE_ERR_PLAN_INFEASIBLE;
    if (plan->co_warps < 0 || plan->co_warps > kCoWarpsMax) return MOE_ERR_PLAN_INFEASIBLE;
    if (mode != MOE_MODE_COMBINE_ONLY && Pc < 1) return MOE_ERR_PLAN_INFEASIBLE;
    if (mode == MOE_MODE_FUSED && (int64_t)plan->R * o_comm < C) return MOE_ERR_PLAN_INFEASIBLE;
    // every CTA must be resident at once: spinning communication CTAs may never keep a compute
    // CTA off the GPU (Section II-C: the legal set keeps positive compute capacity)
    if (ceil_div(C, o_comm) + ceil_div(Pc, o_comp) * slot_sms > h->G) return MOE_ERR_PLAN_INFEASIBLE;
    if (pair && (((C + 1) & ~1) + 2 * Pc > 2 * h->max_pairs)) return MOE_ERR_PLAN_INFEASIBLE;
    if (const int32_t rc = require_handle_device(h, "moe_gemm2_combine")) return rc;

    FusedParams p;
    memset(&p, 0, sizeof p);
    const int K = s->I / s->TP;
    const int TN = occ->tile_n;
    p.T = s->T; p.H = s->H; p.K = K; p.TP = s->TP; p.EP = s->EP; p.L = s->L; p.k_tot = s->k_tot;
    p.S = n_mtiles;
    p.tile_m = occ->tile_m;
    p.flag_parts = pair ? 2 : 1;
    p.split_w = (int32_t)ceil_div(s->H, s->L);
    p.NTs = (int32_t)ceil_div(p.split_w, TN);
    const int64_t Wc = (int64_t)s->TP * n_mtiles * p.NTs;
    if (Wc * s->L * 2 >= (int64_t)1 << 31) return MOE_ERR_SHAPE;
    p.W_comp = (int32_t)Wc;
    p.S_dev = counts_on_device ? r->tiles + s->E_tot : nullptr;
    p.C = C; p.P = Pc; p.mode = mode; p.withhold = plan->debug_withhold_tile;
    p.drain_help = (mode == MOE_MODE_FUSED && plan->drain_help) ? 1 : 0;
    p.tok_blk = (int32_t)ceil_div(s->T, s->EP);
    p.tok_tiles_per_rank = (int32_t)ceil_div(p.tok_blk, kCommTileM);
    p.comm_cols = (int32_t)ceil_div(p.split_w, kCommTileN);
    int64_t tok_tiles = 0;
    for (int d = 0; d < s->EP; ++d) {
        int64_t own = (int64_t)s->T - (int64_t)d * p.tok_blk;
        if (own > p.tok_blk) own = p.tok_blk;
        if (own > 0) tok_tiles += ceil_div(own, kCommTileM);
    }
    p.comm_tiles = (int32_t)(tok_tiles * p.comm_cols);
    p.num_kb = (int32_t)ceil_div(K, kBlockK);
    p.last_ksteps = (K - (p.num_kb - 1) * kBlockK) / kUmmaK;
    p.R_pad = (long long)occ->tile_m * n_mtiles;
    p.wait_ns = h->wait_ns;
    p.mtile_expert = r->mtile_expert;
    p.mtile_first_row = r->mtile_first_row;
    p.mtile_valid = r->mtile_valid;
    p.pad_row = r->pad_row;
    p.perm = r->perm;
    p.Q = s->k_tot * s->TP;
    {   // column slab of one unit: the largest power of two with Q * slab_cols * 2 <= 8 KB, at most 1024
        int sh = 10;
        while (sh > 3 && ((int64_t)p.Q << sh) * 2 > 8192) --sh;
        p.slab_shift = sh;
        p.slab_cols = 1 << sh;
    }
    p.topk_w = topk_w;
    p.Y = y_ws;
    p.wide_store = (p.slab_cols >= 32 && p.split_w % 16 == 0 && s->H % 16 == 0 &&
                    (reinterpret_cast<uintptr_t>(y_ws) & 31u) == 0) ? 1 : 0;
    p.status = status_dev;
    for (int d = 0; d < s->EP; ++d) p.out[d] = out[d];
    // Co-resident communication warps need the dynamic hand-out (they pull from the queues), the aux region
    // of shared memory (free only when the epilogue stores straight from registers) and units of at most 16
    // rows; where one of these does not hold the launch runs without them (same result, bit for bit).
    p.co_warps = plan->co_warps < fused_co_warps_max() ? plan->co_warps : fused_co_warps_max();
    if (!p.drain_help || !p.wide_store || p.Q > 16) p.co_warps = 0;
    // warps 16-19 of a compute CTA: co-resident communication warps, or -- when none is asked for -- a fourth
    // epilogue column group (a third less epilogue work per warp: what bounds tiles with a short K)
    p.epi_warps = (p.co_warps == 0 && p.wide_store) ? 16 : 12;
    // CTA-pair kernel: with the aux region free during the GEMM it becomes a seventh operand stage
    p.pair_stages = (pair && p.co_warps == 0 && p.wide_store && kPairSeventhStage) ? 7 : 6;
    // Tile sequence: split-major (the paper's) whenever something consumes a split while the next one is
    // computed; m-tile-major across the splits (x is read from DRAM once) when nothing does
    p.tile_order = (plan->drain_help && p.co_warps == 0) ? 1 : 0;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    // launch epoch of this workspace: a flag equal to the epoch means "ready in this launch"
    uint32_t &ep = h->epochs[flags_ws];
    ep += 1u;
    if (ep == 0u) {  // wrapped: start over from a clean workspace
        size_t fb = 0;
        moe_workspace_bytes(s, occ->tile_m, occ->tile_n, nullptr, nullptr, &fb, nullptr);
        e = cudaMemsetAsync(flags_ws, 0, fb - 16, st);
        if (e != cudaSuccess) return cuda_fail(h, e, "flags reset");
        ep = 1u;
    }
    p.epoch = ep;
    p.split_done = flags_ws + (ep & 1u) * MOE_MAX_L;
    p.split_done_next = flags_ws + ((ep + 1u) & 1u) * MOE_MAX_L;
    p.queue = reinterpret_cast<unsigned long long *>(flags_ws + 2 * MOE_MAX_L) + (ep & 1u) * MOE_MAX_L;
    p.queue_next = reinterpret_cast<unsigned long long *>(flags_ws + 2 * MOE_MAX_L) + ((ep + 1u) & 1u) * MOE_MAX_L;
    p.flags = flags_ws + kSplitCounterWords;

    // tensor maps (Section II-A operands): x_routed [R, I] and W2 [E_tot, H, I], k contiguous.  Encoding the two
    // maps costs microseconds of host time between the wait for the tile counts and the launch: the handle
    // keeps the last pair and reuses it while buffers, sizes and tile family stay the same (a loop of steps).
    const TensorMapKey key = {x_routed, W2, s->T, s->k_tot, s->I, s->H, s->E_tot, pair ? TN / 2 : TN};
    if (!h->tm_valid || memcmp(&h->tm_key, &key, sizeof key) != 0) {
        EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(h->encode_tiled);
        const cuuint64_t R = (cuuint64_t)s->T * s->k_tot;
        h->tm_valid = false;
        {
            cuuint64_t dims[2] = {(cuuint64_t)s->I, R};
            cuuint64_t strides[1] = {(cuuint64_t)s->I * 2};
            cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)kMmaM};
            cuuint32_t es[2] = {1, 1};
            CUresult cr = encode(&h->tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(x_routed), dims,
                                 strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (cr != CUDA_SUCCESS) {
                snprintf(h->err, sizeof h->err, "cuTensorMapEncodeTiled(x_routed) failed: %d", (int)cr);
                return MOE_ERR_CUDA;
            }
        }
        {
            cuuint64_t dims[3] = {(cuuint64_t)s->I, (cuuint64_t)s->H, (cuuint64_t)s->E_tot};
            cuuint64_t strides[2] = {(cuuint64_t)s->I * 2, (cuuint64_t)s->H * s->I * 2};
            cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)(pair ? TN / 2 : TN), 1};   // a pair CTA loads half the rows
            cuuint32_t es[3] = {1, 1, 1};
            CUresult cr = encode(&h->tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(W2), dims, strides,
                                 box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (cr != CUDA_SUCCESS) {
                snprintf(h->err, sizeof h->err, "cuTensorMapEncodeTiled(W2) failed: %d", (int)cr);
                return MOE_ERR_CUDA;
            }
        }
        h->tm_key = key;
        h->tm_valid = true;
    }
    p.tmA = h->tmA;
    p.tmB = h->tmB;
    const int grid = pair ? ((C + 1) & ~1) + 2 * Pc : C + Pc;
    p.timeline = nullptr;
    if (h->timeline && h->timeline_bytes >= ((size_t)grid * kTimelineSlots + MOE_MAX_L) * sizeof(unsigned long long))
        p.timeline = h->timeline;
    p.probe = h->probe;
    e = pair ? pair_launch(p, grid, st) : fused_launch(TN, p, grid, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "fused launch");
    return MOE_OK;
}

int32_t moe_release_workspace(moe_handle *h, const uint32_t *flags_ws)
{
    if (!h) return MOE_ERR_NULL;
    if (flags_ws) h->epochs.erase(flags_ws);
    else h->epochs.clear();
    return MOE_OK;
}

int32_t moe_get_status(moe_handle *h, const uint32_t *status_dev, moe_status *host, void *stream)
{
    if (!h || !status_dev || !host) return MOE_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t w[4];
    cudaError_t e = cudaMemcpyAsync(w, status_dev, sizeof w, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(h, e, "status copy");
    host->code = w[0]; host->detail = w[1]; host->where = w[2]; host->count = w[3];
    return w[0] == 0 ? MOE_OK : MOE_ERR_DEVICE_STATUS;
}

int32_t moe_clear_status(moe_handle *h, uint32_t *status_dev, void *stream)
{
    if (!h || !status_dev) return MOE_ERR_NULL;
    cudaError_t e = cudaMemsetAsync(status_dev, 0, 16, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MOE_OK : cuda_fail(h, e, "status clear");
}

// ---- whole step on device-resident inputs -----------------------------------------------------

int32_t moe_layer(moe_handle *h, const void *x_routed, const void *W2, const int32_t *topk_idx,
                  const float *topk_w, const moe_shape *s, int32_t tile_m, int32_t tile_n,
                  const moe_sm_limits *limits_or_null, const moe_routing *routing,
                  int32_t *tile_counts_pinned, void *const *out, void *y_ws, uint32_t *flags_ws,
                  uint32_t *status_dev, moe_plan *plan_out, void *ev_before, void *ev_after, void *stream)
{
    if (!h || !s || !routing) return MOE_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t seq = 0;
    int32_t rc = build_routing_mailed(h, topk_idx, s, tile_m, routing, tile_counts_pinned, status_dev, st, &seq);
    if (rc != MOE_OK) return rc;
    if (tile_counts_pinned) {
        // the counts reach the host while the routing build is still scattering: planning and the fused
        // launch below are queued behind it without a gap
        rc = wait_counts(h, seq, s->E_tot, tile_counts_pinned, st, nullptr);
        if (rc != MOE_OK) return rc;
    }
    moe_occupancy occ;
    moe_sm_limits lim;
    moe_rho rho;
    rc = moe_query_occupancy(h, tile_m, tile_n, &occ, &lim, &rho);
    if (rc != MOE_OK) return rc;
    if (limits_or_null) lim = *limits_or_null;
    moe_plan plan;
    rc = tile_counts_pinned ? plan_partition(tile_counts_pinned, s->E_tot, &occ, &lim, s, &rho, &plan)
                            : plan_partition_estimate(&occ, &lim, s, &rho, &plan);   // counts stay on the device
    if (rc != MOE_OK) return rc;
    if (plan_out) *plan_out = plan;
    if (ev_before) cudaEventRecord(static_cast<cudaEvent_t>(ev_before), st);
    rc = moe_gemm2_combine(h, x_routed, W2, topk_idx, topk_w, s, &occ, routing,
                           tile_counts_pinned ? tile_counts_pinned[s->E_tot] : MOE_MTILES_ON_DEVICE, &plan,
                           out, y_ws, flags_ws, status_dev, st);
    if (ev_after) cudaEventRecord(static_cast<cudaEvent_t>(ev_after), st);
    return rc;
}

// ---- the post-router MoE layer on device-resident inputs (Section II-A: steps 1-3) -------------

int32_t moe_post_router_layer(moe_handle *h, const void *hidden, const void *W1, const void *W2,
                              const int32_t *topk_idx, const float *topk_w, const moe_shape *s, int32_t tile_m,
                              int32_t tile_n, const moe_sm_limits *limits_or_null, const moe_routing *routing,
                              int32_t *tile_counts_pinned, void *h_routed_ws, void *x_routed_ws, void *const *out,
                              void *y_ws, uint32_t *flags_ws, uint32_t *status_dev, moe_plan *plan_out, void *stream)
{
    if (!h || !s || !routing) return MOE_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t seq = 0;
    int32_t rc = build_routing_mailed(h, topk_idx, s, tile_m, routing, tile_counts_pinned, status_dev, st, &seq);
    if (rc != MOE_OK) return rc;
    // GEMM1 reads the m-tile count on the device, so it is launched before the host waits for the counts:
    // the wait and the planning are hidden behind it
    if (tile_counts_pinned && seq == 0u && h->counts_event) cudaEventRecord(static_cast<cudaEvent_t>(h->counts_event), st);
    rc = moe_gemm1_act(h, hidden, W1, s, tile_m, routing, MOE_MTILES_ON_DEVICE, h_routed_ws, x_routed_ws, status_dev, st);
    if (rc != MOE_OK) return rc;
    moe_occupancy occ;
    moe_sm_limits lim;
    moe_rho rho;
    rc = moe_query_occupancy(h, tile_m, tile_n, &occ, &lim, &rho);
    if (rc != MOE_OK) return rc;
    if (limits_or_null) lim = *limits_or_null;
    moe_plan plan;
    int32_t n_mtiles = MOE_MTILES_ON_DEVICE;
    if (tile_counts_pinned) {
        // the copy of the counts was queued right after the routing kernels, before GEMM1: wait for it alone
        cudaEvent_t counts_ready = static_cast<cudaEvent_t>(h->counts_event);
        if (seq == 0u && !counts_ready) return MOE_ERR_CUDA;
        rc = wait_counts(h, seq, s->E_tot, tile_counts_pinned, st, counts_ready);
        if (rc != MOE_OK) return rc;
        rc = plan_partition(tile_counts_pinned, s->E_tot, &occ, &lim, s, &rho, &plan);
        n_mtiles = tile_counts_pinned[s->E_tot];
    } else {
        rc = plan_partition_estimate(&occ, &lim, s, &rho, &plan);
    }
    if (rc != MOE_OK) return rc;
    if (plan_out) *plan_out = plan;
    return moe_gemm2_combine(h, x_routed_ws, W2, topk_idx, topk_w, s, &occ, routing, n_mtiles, &plan, out, y_ws,
                             flags_ws, status_dev, st);
}

// ---- one-time service-rate characterisation (Eq. 13) ---------------------------------------

int32_t moe_calibrate_rho(moe_handle *h, const void *x_routed, const void *W2, const int32_t *topk_idx,
                          const float *topk_w, const moe_shape *s, int32_t tile_m, int32_t tile_n,
                          int32_t C_ref, int32_t n_samples, const moe_routing *routing,
                          int32_t *tile_counts_pinned, void *const *out, void *y_ws, uint32_t *flags_ws,
                          uint32_t *status_dev, moe_rho *rho_out, double *wave_us_out, void *stream)
{
    if (!h || !s || !routing || !tile_counts_pinned || !rho_out) return MOE_ERR_NULL;
    if (C_ref < 1 || n_samples < 1 || n_samples > 64) return MOE_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t rc = moe_build_routing(h, topk_idx, s, tile_m, routing, tile_counts_pinned, status_dev, st);
    if (rc != MOE_OK) return rc;
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(h, e, "tile counts sync");
    moe_occupancy occ;
    moe_sm_limits lim;
    moe_rho rho;
    rc = moe_query_occupancy(h, tile_m, tile_n, &occ, &lim, &rho);
    if (rc != MOE_OK) return rc;
    lim.force_comm_ctas = C_ref;
    lim.drain_help = 0;                       // each role alone on its share of the SMs
    moe_plan plan;
    rc = plan_partition(tile_counts_pinned, s->E_tot, &occ, &lim, s, &rho, &plan);
    if (rc != MOE_OK) return rc;
    if (plan.W_comp < 1 || plan.W_comm < 1) return MOE_ERR_SHAPE;
    const int32_t S = tile_counts_pinned[s->E_tot];

    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    if ((e = cudaEventCreate(&ev0)) != cudaSuccess) return cuda_fail(h, e, "event");
    if ((e = cudaEventCreate(&ev1)) != cudaSuccess) { cudaEventDestroy(ev0); return cuda_fail(h, e, "event"); }
    double med[2] = {0.0, 0.0};
    for (int role = 0; role < 2 && rc == MOE_OK; ++role) {
        moe_plan p = plan;
        p.mode = role == 0 ? MOE_MODE_GEMM_ONLY : MOE_MODE_COMBINE_ONLY;   // GEMM first: it also fills Y
        float t[64];
        for (int i = -2; i < n_samples && rc == MOE_OK; ++i) {              // two warm-up launches
            cudaEventRecord(ev0, st);
            rc = moe_gemm2_combine(h, x_routed, W2, topk_idx, topk_w, s, &occ, routing, S, &p, out, y_ws,
                                   flags_ws, status_dev, st);
            cudaEventRecord(ev1, st);
            if ((e = cudaEventSynchronize(ev1)) != cudaSuccess) rc = cuda_fail(h, e, "calibration launch");
            if (rc == MOE_OK && i >= 0) cudaEventElapsedTime(&t[i], ev0, ev1);
        }
        if (rc == MOE_OK) {
            std::sort(t, t + n_samples);
            med[role] = 1e3 * (double)t[n_samples / 2];
        }
    }
    cudaEventDestroy(ev0);
    cudaEventDestroy(ev1);
    if (rc != MOE_OK) return rc;
    // Eq. 13: time per wave of each role; a launch runs L splits of V waves each
    const double comp_waves = (double)ceil_div(plan.W_comp, plan.P) * s->L;
    const double comm_waves = (double)ceil_div(plan.W_comm, C_ref) * s->L;
    const double wave_comp = med[0] / comp_waves, wave_comm = med[1] / comm_waves;
    if (!(wave_comp > 0.0)) return MOE_ERR_SHAPE;
    if (wave_us_out) { wave_us_out[0] = wave_comp; wave_us_out[1] = wave_comm; }
    *rho_out = rho;
    rho_out->rho_ref = wave_comm / wave_comp;
    rho_out->K_ref = s->I / s->TP;
    rho_out->tile_m_ref = tile_m;
    rho_out->tile_n_ref = tile_n;
    rho_out->D_ref = s->EP;
    rho_out->rows_ref = s->k_tot * s->TP + 1;
    const int64_t split_w = ceil_div(s->H, s->L);
    rho_out->comm_cols_ref = (int32_t)(split_w < kCommTileN ? split_w : kCommTileN);
    return MOE_OK;
}

// ---- whole step from host buffers ----------------------------------------------------------

namespace {
struct ArenaLayout {
    size_t x, idx, w, routing, y, flags, status, out, total;
    size_t routing_b, y_b, flags_b;
};
int32_t arena_layout(const moe_shape *s, int tile_m, int tile_n, ArenaLayout *a)
{
    size_t sb = 0;
    int32_t rc = moe_workspace_bytes(s, tile_m, tile_n, &a->routing_b, &a->y_b, &a->flags_b, &sb);
    if (rc != MOE_OK) return rc;
    const size_t R = (size_t)s->T * s->k_tot;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    size_t off = 0;
    a->x = off; off += up(R * s->I * 2);
    a->idx = off; off += up(R * 4);
    a->w = off; off += up(R * 4);
    a->routing = off; off += up(a->routing_b);
    a->y = off; off += up(a->y_b);
    a->flags = off; off += up(a->flags_b);
    a->status = off; off += up(16);
    a->out = off; off += up((size_t)ceil_div(s->T, s->EP) * s->EP * s->H * 2);
    a->total = off;
    return MOE_OK;
}
}  // namespace

int32_t moe_host_arena_bytes(const moe_shape *s, int32_t tile_m, int32_t tile_n, size_t *bytes)
{
    if (!s || !bytes) return MOE_ERR_NULL;
    ArenaLayout a;
    int32_t rc = arena_layout(s, tile_m, tile_n, &a);
    if (rc != MOE_OK) return rc;
    *bytes = a.total;
    return MOE_OK;
}

int32_t moe_layer_host(moe_handle *h, const void *x_routed_host, const int32_t *topk_idx_host,
                       const float *topk_w_host, const void *W2_dev, const moe_shape *s, int32_t tile_m,
                       int32_t tile_n, const moe_sm_limits *limits_or_null, void *arena, size_t arena_bytes,
                       int32_t *tile_counts_pinned, void *out_host, moe_plan *plan_out, void *stream)
{
    if (!h || !s || !arena || !tile_counts_pinned || !out_host || !W2_dev) return MOE_ERR_NULL;
    if (s->T > 0 && (!x_routed_host || !topk_idx_host || !topk_w_host)) return MOE_ERR_NULL;
    ArenaLayout a;
    int32_t rc = arena_layout(s, tile_m, tile_n, &a);
    if (rc != MOE_OK) return rc;
    if (arena_bytes < a.total) return MOE_ERR_ARENA;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return MOE_ERR_ALIGN;
    if (s->T == 0) return MOE_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *base = static_cast<char *>(arena);
    const size_t R = (size_t)s->T * s->k_tot;
    cudaError_t e;
    e = cudaMemcpyAsync(base + a.idx, topk_idx_host, R * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(base + a.status, 0, 16, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "idx copy");
    moe_routing rt;
    rc = moe_routing_view(base + a.routing, s, tile_m, &rt);
    if (rc != MOE_OK) return rc;
    uint32_t *status = reinterpret_cast<uint32_t *>(base + a.status);
    rc = moe_build_routing(h, reinterpret_cast<int32_t *>(base + a.idx), s, tile_m, &rt, tile_counts_pinned,
                           status, st);
    if (rc != MOE_OK) return rc;
    cudaEvent_t counts_ready;
    e = cudaEventCreateWithFlags(&counts_ready, cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(h, e, "event");
    cudaEventRecord(counts_ready, st);
    // the large copies overlap the wait for the counts
    e = cudaMemcpyAsync(base + a.x, x_routed_host, R * s->I * 2, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(base + a.w, topk_w_host, R * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(base + a.flags, 0, a.flags_b, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(counts_ready);
    cudaEventDestroy(counts_ready);
    if (e != cudaSuccess) return cuda_fail(h, e, "input copies");
    h->epochs.erase(base + a.flags);  // the workspace was just cleared

    moe_occupancy occ;
    moe_sm_limits lim;
    moe_rho rho;
    rc = moe_query_occupancy(h, tile_m, tile_n, &occ, &lim, &rho);
    if (rc != MOE_OK) return rc;
    if (limits_or_null) lim = *limits_or_null;
    moe_plan plan;
    rc = plan_partition(tile_counts_pinned, s->E_tot, &occ, &lim, s, &rho, &plan);
    if (rc != MOE_OK) return rc;
    if (plan_out) *plan_out = plan;
    void *outs[MOE_MAX_EP];
    const size_t blk = (size_t)ceil_div(s->T, s->EP);
    for (int d = 0; d < s->EP; ++d) outs[d] = base + a.out + (size_t)d * blk * s->H * 2;
    rc = moe_gemm2_combine(h, base + a.x, W2_dev, nullptr, reinterpret_cast<float *>(base + a.w), s, &occ, &rt,
                           tile_counts_pinned[s->E_tot], &plan, outs, base + a.y,
                           reinterpret_cast<uint32_t *>(base + a.flags), status, st);
    if (rc != MOE_OK) return rc;
    // rank d owns tokens [d*blk, (d+1)*blk): the EP blocks are contiguous in token order
    e = cudaMemcpyAsync(out_host, base + a.out, (size_t)s->T * s->H * 2, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(h, e, "output copy");
    moe_status hs;
    return moe_get_status(h, status, &hs, st);
}

}  // extern "C"
