/*
 * moe_b200.h -- C ABI of the B200 (sm_100a) MoE down-projection operator:
 * grouped expert GEMM2 fused with the GatherRS combine, plus the launch-time analytical
 * selector of the communication-CTA count.
 *
 * Citations name sections / equations / algorithms of the paper
 * "Analytical Resource Management for Fine-grained MoE Computation-Communication Overlap".
 *
 * Conventions
 *  - every function returns an int32 status: MOE_OK (0) or a negative MOE_ERR_* value;
 *    nothing throws across this boundary;
 *  - pointers are tagged [host] or [device]; the library never allocates device memory:
 *    the caller owns every buffer and the stream (passed as void*, a cudaStream_t);
 *  - all launches are asynchronous on the given stream; the handle's device must be the calling
 *    thread's current CUDA device (checked by every launching call: MOE_ERR_UNSUPPORTED otherwise);
 *  - a handle is not thread-safe: one host thread uses it at a time (it keeps the text of the last
 *    error and the launch epoch of every flags workspace it has launched on);
 *  - device-side problems (a bounded wait that ran out, an index out of range) are reported
 *    through a 4-word status buffer in device memory, read back with moe_get_status();
 *  - bf16 tensors are passed as void*; layouts are row-major with the last index contiguous.
 *
 * Symbols: T tokens (paper M), H hidden size (paper N), I expert intermediate size,
 * TP emulated tensor-parallel shards (split-K partials, paper g), K = I / TP (paper K),
 * EP emulated destination ranks (paper D), E_tot experts (routed + shared), k_tot experts per
 * token, R = T * k_tot routed rows, L pipeline splits along H, S = sum_e ceil(M_e / T_M).
 */
#ifndef MOE_B200_H
#define MOE_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    MOE_OK = 0,
    MOE_ERR_NULL = -1,            /* a required pointer is NULL */
    MOE_ERR_SHAPE = -2,           /* unsupported or inconsistent sizes */
    MOE_ERR_ALIGN = -3,           /* a device pointer is not 16-byte aligned */
    MOE_ERR_PLAN_INFEASIBLE = -4, /* no legal C, or the plan does not fit the GPU */
    MOE_ERR_CUDA = -5,            /* a CUDA runtime/driver call failed (see moe_last_cuda_error) */
    MOE_ERR_UNSUPPORTED = -6,     /* tile configuration the kernels do not provide */
    MOE_ERR_DEVICE_STATUS = -7,   /* the device status buffer reports a problem */
    MOE_ERR_ARENA = -8,           /* the caller's arena is too small */
    MOE_ERR_STATIC_LIMIT = -9     /* the problem needs more scratch than the built-in array holds */
};

/* device status codes (word 0 of the status buffer) */
enum {
    MOE_DEV_OK = 0,
    MOE_DEV_TIMEOUT = 1,   /* a bounded wait ran out; word 1 = tile / flag index, word 2 = where */
    MOE_DEV_OOB = 2,       /* an index was out of range and the access was skipped; word 1 = index */
    MOE_DEV_DUP_EXPERT = 3 /* one token names the same expert twice; word 1 = token */
};

enum { MOE_MODE_FUSED = 0, MOE_MODE_GEMM_ONLY = 1, MOE_MODE_COMBINE_ONLY = 2 };
/* MOE_RHO_PAPER: Eq. 14 as printed (K, tile area and D/D_ref terms).
 * MOE_RHO_LOCAL: the re-derivation Section III-E asks of a new kernel family, for ranks
 * emulated inside one GPU: no ring term D/D_ref; a communication tile costs in proportion
 * to the rows it moves per token (k_tot * TP read + 1 written) and to its real width
 * min(T_N^comm, ceil(H/L)). */
enum { MOE_RHO_PAPER = 0, MOE_RHO_LOCAL = 1 };
enum { MOE_DEP_SPLIT = 0, MOE_DEP_TILE = 1 };
#define MOE_MAX_EP 8
#define MOE_MAX_L 8
#define MOE_MTILES_ON_DEVICE (-1)   /* moe_gemm2_combine: read the m-tile count from routing->tiles[E_tot] on the device */

typedef struct moe_handle moe_handle;

typedef struct {
    int32_t T, H, I, E_tot, k_tot, TP, EP, L;
} moe_shape;

/* Kernel-family constants of one GEMM2 tile configuration (Section III-B, Table I; Section
 * III-E: read once per kernel choice, not per invocation). */
typedef struct {
    int32_t tile_m, tile_n;           /* T_M^comp, T_N^comp */
    int32_t comm_tile_m, comm_tile_n; /* T_M^comm, T_N^comm */
    int32_t o_comp, o_comm;           /* resident CTAs per SM of each role */
    int32_t comp_slot_sms;            /* SMs one compute slot occupies: 1, or 2 when a compute tile is run
                                         by a pair of CTAs on two SMs; P(C) = o_comp * floor((G - R(C)) / comp_slot_sms) */
} moe_occupancy;

/* GPU residency limits and the user's overrides (Section III-D legal set; Section III-E:
 * an explicit C has the highest priority, and the selector can be switched off). */
typedef struct {
    int32_t G;               /* SMs available to the operator */
    int32_t C_max;           /* upper end of the legal set {1..C_max} */
    int32_t force_comm_ctas; /* > 0: use exactly this C */
    int32_t selector_off;    /* != 0: use default_C */
    int32_t default_C;       /* the fixed count used when the selector is off */
    int32_t drain_help;      /* != 0: compute CTAs that run out of GEMM tiles serve the communication work
                                that is left, and the work is handed out dynamically (warps pull token ranges
                                from a queue per split) instead of by the static tile -> CTA map (an extension
                                of this library, not in the paper: with it the selector models the tail after
                                the last compute wave as served by every SM);
                                0: the paper's static partition and its recurrence exactly */
    int32_t co_warps_max;    /* upper end of the legal set {0..co_warps_max} of co-resident communication warps
                                per compute CTA (0: a kernel family without them) */
    int32_t force_co_warps;  /* >= 0: use exactly this many (clamped to co_warps_max); < 0: the selector decides */
    int32_t C_co_max;        /* dedicated communication CTAs tried beside co-resident warps: C in 1..min(C_max, C_co_max)
                                for w >= 1 (a one-time characterisation, like C_max) */
    int32_t dep_model;       /* static partition only: MOE_DEP_SPLIT = Eq. 9 as printed (one readiness per split),
                                MOE_DEP_TILE = Eq. 9 applied to every communication tile (per-tile flags) */
    int32_t co_min_waves;    /* lower end of the legal set for co-resident warps: they are tried only when the compute
                                phase is at least this many waves long, ceil(L * W_comp / P(C)) >= co_min_waves (a
                                one-time characterisation: on short launches their start-up costs more than they can
                                overlap; moe_query_occupancy returns INT32_MAX for the 256-row CTA-pair tiles, where
                                a co-resident warp costs the seventh operand stage and never paid); a forced w is not
                                subject to it */
} moe_sm_limits;

/* Relative wave service rate (Eq. 13-15). */
typedef struct {
    double rho_ref;
    int32_t K_ref, tile_m_ref, tile_n_ref, D_ref;
    int32_t rows_ref;        /* k_tot * TP + 1 of the reference run (MOE_RHO_LOCAL only) */
    int32_t comm_cols_ref;   /* min(T_N^comm, ceil(H/L)) of the reference run (MOE_RHO_LOCAL only) */
    int32_t mode;            /* MOE_RHO_PAPER | MOE_RHO_LOCAL */
    /* Bandwidth coupling and co-resident communication warps (this library's re-derivation for a kernel
     * family whose communication work can share SMs with compute; used with drain_help only; all zero =
     * the plain recurrence).  Capacity is counted in warps: a communication tile is comm_warps_per_cta
     * quanta, a dedicated communication CTA serves comm_warps_per_cta of them per wave. */
    int32_t comm_warps_per_cta; /* warps of a communication CTA (0: coupling and co-resident warps off) */
    int32_t n_sat_warps;        /* warps streaming together that saturate HBM: above it one quantum takes
                                   rho * N / n_sat_warps (0: never saturated) */
    int32_t comm_quanta_per_tile; /* pieces a communication tile is handed out in (0: one per warp of a CTA; the
                                   dynamic hand-out gives out single tokens: T_M^comm); one warp serves a piece in
                                   rho * comm_warps_per_cta / comm_quanta_per_tile */
    int32_t reserved0;
    double co_beta;             /* one co-resident warp stretches the compute wave by this fraction */
    double co_gamma;            /* a co-resident warp serves this many times slower than a dedicated one (>= 1) */
    double co_order;            /* with co-resident warps and L > 1 the tile order is split-major (x is read once
                                   per split): the compute wave is stretched by this fraction */
} moe_rho;

/* Result of the selector, and the launch description moe_gemm2_combine() consumes.
 * Plain data: the caller may overwrite comm_ctas / R / P (validated at launch). */
typedef struct {
    int32_t comm_ctas;   /* C*   */
    int32_t R;           /* R(C*) = ceil(C / o_comm), SM positions reserved (Eq. 1) */
    int32_t P;           /* P(C*) = o_comp floor((G - R) / comp_slot_sms), compute slots (Eq. 3) */
    int32_t W_comp;      /* Eq. 5, compute tiles per split */
    int32_t W_comm;      /* communication tiles per split on this GPU (Eq. 7 summed over ranks) */
    int32_t delta;       /* Delta_comp(C*) (tie breaker) */
    int64_t pred_T_q;    /* T(C*) in compute-wave units, scaled by 2^20 */
    int64_t rho_q;       /* rho scaled by 2^20 and rounded to nearest */
    int32_t mode;        /* MOE_MODE_* (plan_partition writes MOE_MODE_FUSED) */
    int32_t debug_withhold_tile; /* test hook: global tile whose readiness is never raised; -1 = none */
    int32_t drain_help;  /* copied from moe_sm_limits: compute CTAs help with the communication tail */
    int32_t co_warps;    /* co-resident communication warps per compute CTA (Section III-B with communication
                            work sharing the SM of a compute CTA instead of reserving one): they serve split s
                            while the CTA computes split s + 1.  Needs drain_help; the launch drops them when
                            the shape leaves them no shared memory (see moe_gemm2_combine) */
} moe_plan;

/* Views into the routing workspace, all [device] int32. */
typedef struct {
    int32_t *counts;          /* [E_tot]     M_e */
    int32_t *offsets;         /* [E_tot + 1] exclusive prefix of counts */
    int32_t *tiles;           /* [E_tot + 1] ceil(M_e / T_M), then S */
    int32_t *tile_offsets;    /* [E_tot + 1] exclusive prefix of tiles; last = S */
    int32_t *perm;            /* [R] flat assignment held by routed row r */
    int32_t *inv_perm;        /* [R] routed row of flat assignment f = t * k_tot + j */
    int32_t *pad_row;         /* [R] row of f in the tile-padded layout */
    int32_t *mtile_expert;    /* [max_mtiles] */
    int32_t *mtile_first_row; /* [max_mtiles] */
    int32_t *mtile_valid;     /* [max_mtiles] */
    int32_t *scratch;         /* per-warp histograms used while building */
    int32_t max_mtiles;       /* floor(R / T_M) + E_tot, an upper bound of S */
} moe_routing;

typedef struct {
    uint32_t code, detail, where, count;
} moe_status;

/* ---- handle -------------------------------------------------------------------------- */

/* Opens the library on CUDA device `device`; caches the SM count and the kernels'
 * residency (Section III-E: the SM count is cached at operator initialisation).  Also allocates the
 * handle's only memory outside the C++ heap: about 4 KB of pinned host memory that the GPU can address,
 * the mailbox through which the routing build hands the routed-tile counts to the whole-step calls
 * (moe_layer, moe_post_router_layer); freed by moe_destroy.  No device memory is allocated.  [host] */
int32_t moe_create(int32_t device, moe_handle **out);
int32_t moe_destroy(moe_handle *h);
/* Text of the last failing CUDA call on this handle ("" if none); owned by the handle. */
const char *moe_last_cuda_error(const moe_handle *h);
/* Upper bound, in nanoseconds, of every device-side wait (default 2e9).  After it a CTA
 * records MOE_DEV_TIMEOUT and leaves; the context stays usable.  The limit is counted from
 * the start of each CTA, so it bounds the whole launch as well. */
int32_t moe_set_wait_limit_ns(moe_handle *h, uint64_t ns);

/* Tracing aid (Section III-C characterises service rates by timing the two roles; this is the tool for
 * it).  In a library built with -DMOE_TIMELINE=1 (python -m paper_2609_07536_b200.build --timeline, a
 * separate libmoe_b200_timeline.so) every later moe_gemm2_combine launch on this handle records, per CTA,
 * MOE_TIMELINE_SLOTS 64-bit words -- %globaltimer stamps (CTA begin, first accumulator, last MMA, end of
 * the compute role, CTA end), cycle counters of the MMA-issuing thread (waiting for operands, issuing,
 * waiting for an accumulator buffer), of one epilogue warp and of one producer, and what its communication
 * warps served and when -- followed by one completion stamp per split, into timeline_dev [device, 8-byte
 * aligned, at least (grid * MOE_TIMELINE_SLOTS + MOE_MAX_L) * 8 bytes, zero-filled by the caller; a buffer
 * that is too small for a launch is left alone].  NULL switches recording off.  The normal library accepts
 * only NULL (MOE_ERR_UNSUPPORTED otherwise): its kernels carry no instrumentation.  bench.py --timeline
 * reads the records.  [host] */
#define MOE_TIMELINE_SLOTS 40
int32_t moe_set_timeline(moe_handle *h, void *timeline_dev, size_t bytes);
/* Timeline build only: later fused launches on this handle leave out part of their data movement, so that its
 * cost shows in the launch time (the outputs of such a launch are garbage by construction; never for a result
 * that is used).  Bits: MOE_PROBE_SKIP_ODD_W2 (the W2 tile of every second k-block is not loaded: a quarter
 * less operand traffic), MOE_PROBE_SKIP_ALL_W2 (no W2 tile is loaded: half the operand traffic),
 * MOE_PROBE_SKIP_Y_STORES (the epilogue converts but does not store: no Y write traffic; GEMM-only launches),
 * MOE_PROBE_SKIP_X (256-row pair tiles: no x_routed tile is loaded; with MOE_PROBE_SKIP_ALL_W2 the MMAs run on
 * whatever shared memory holds and the launch time is that of MMA issue and epilogue alone),
 * MOE_PROBE_FREE_RUN_MMA (256-row pair tiles: no loads, no operand barriers, no per-k-block commit: the rate at
 * which the tensor pipe takes the MMAs when nothing but the accumulator hand-over gates them),
 * MOE_PROBE_SLOW_ISSUER (256-row pair tiles: the thread that issues the MMAs idles 200 cycles per k-block;
 * what the launch loses shows how little the tensor pipe buffers ahead of that thread).
 * 0 switches the probes off; the normal library accepts only 0 (MOE_ERR_UNSUPPORTED otherwise).  [host] */
enum { MOE_PROBE_SKIP_ODD_W2 = 1, MOE_PROBE_SKIP_ALL_W2 = 2, MOE_PROBE_SKIP_Y_STORES = 4, MOE_PROBE_SKIP_X = 8,
       MOE_PROBE_FREE_RUN_MMA = 16, MOE_PROBE_SLOW_ISSUER = 32 };
int32_t moe_set_probe(moe_handle *h, uint32_t probe_bits);

/* Tile shape and residency of the GEMM2 kernel for (tile_m, tile_n), the communication tile,
 * the GPU limits and the stored service-rate constants (Section III-B, III-D, III-E).
 * (tile_m, tile_n): tile_m in {64, 128} with tile_n in {64, 128, 256} (one CTA per tile), or
 * (256, 256) (a pair of CTAs on two SMs per tile).  Any output pointer may be NULL.  [host] */
int32_t moe_query_occupancy(moe_handle *h, int32_t tile_m, int32_t tile_n,
                            moe_occupancy *occ, moe_sm_limits *limits, moe_rho *rho);

/* Kernel dispatch by shape (Section III-E, first paragraph: a conventional dispatch layer selects the GEMM2
 * kernel; the resource manager then reads that kernel's tile shape and residency).  Chooses the GEMM tile
 * family for `shape`: the widest n-tile the split width ceil(H/L) holds (256, 128 or 64), and 256-row
 * CTA-pair tiles when the experts hold at least 192 routed rows on average (T * k_tot / E_tot), 128-row
 * single-CTA tiles below (small and decode-sized token counts: less row padding, every SM its own tile).
 * The result is a valid (tile_m, tile_n) for every other call.  [host] */
int32_t moe_select_tile(moe_handle *h, const moe_shape *shape, int32_t *tile_m, int32_t *tile_n);

/* Sizes of the caller-allocated workspaces [bytes]: routing arrays, the tile-padded GEMM2
 * output Y (bf16, token-major: [T][L][k_tot * TP][ceil(H/L)]), readiness flags + split counters +
 * work queues (must be zero-filled once before first use and not shared between handles), status
 * (16 bytes). */
int32_t moe_workspace_bytes(const moe_shape *shape, int32_t tile_m, int32_t tile_n,
                            size_t *routing_bytes, size_t *y_bytes, size_t *flags_bytes,
                            size_t *status_bytes);
/* Carves the routing workspace [device, 16-byte aligned] into its arrays.  Pure host. */
int32_t moe_routing_view(void *routing_ws, const moe_shape *shape, int32_t tile_m, moe_routing *out);

/* ---- a1: routing / permutation / routed-tile counts ------------------------------------
 * Section II-A (token-expert assignments), Eq. 5 (ceil(M_e / T_M) tiles per expert), Eq. 16
 * (their sum).  Stable sort of the flat assignments f = t * k_tot + j by expert.
 * topk_idx [device] int32 [T, k_tot]; tile_counts_host [host, pinned] receives
 * tiles[0..E_tot) followed by S (E_tot + 1 ints) by an asynchronous copy: synchronise the
 * stream before reading it.  Bad expert ids / repeated experts are reported in status_dev. */
int32_t moe_build_routing(moe_handle *h, const int32_t *topk_idx, const moe_shape *shape,
                          int32_t tile_m, const moe_routing *routing,
                          int32_t *tile_counts_host, uint32_t *status_dev, void *stream);

/* Routing build for callers that cannot allocate device memory (no counterpart in the paper;
 * an addition of this library).  Same inputs, outputs and results as moe_build_routing(), but
 * the builder's scratch (per-warp histograms, ceil(T*k_tot/256) * E_tot ints) lives in a fixed
 * 512 KiB array inside the library instead of routing->scratch, which is ignored and may be
 * NULL.  Meant for code that runs where cudaMalloc is not an option: a serving loop with a
 * memory pool frozen at start-up, a framework allocator that rejects foreign allocations, a
 * latency-critical section that cannot afford the synchronisation an allocation implies.
 * The call itself allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *  - Limit: ceil(T*k_tot/256) * E_tot <= 131072, else MOE_ERR_STATIC_LIMIT (text in
 *    moe_last_cuda_error) and nothing is launched.
 *  - The first call on a device resolves the array's device address (a one-time set-up per
 *    device); make that first call before any stream capture begins.
 *  - All calls on one GPU share the array and it keeps the previous call's contents; the
 *    builder overwrites every entry it later reads, so nothing needs clearing, but two calls
 *    whose kernels overlap on the GPU (different streams) race: order them.
 *  - Every GPU that loads the library holds the 512 KiB until the process exits.
 *  - The handle's device must be the calling thread's current CUDA device, on every call (the array's
 *    address belongs to that device): otherwise MOE_ERR_UNSUPPORTED and nothing is launched. */
int32_t moe_build_routing_static(moe_handle *h, const int32_t *topk_idx, const moe_shape *shape,
                                 int32_t tile_m, const moe_routing *routing,
                                 int32_t *tile_counts_host, uint32_t *status_dev, void *stream);

/* ---- a2: the analytical selector (Section III-D, Algorithm 1, Eq. 1-15, tie breaker) -----
 * Pure host code: no CUDA call, no allocation, re-entrant.
 * routed_tile_counts [host] ceil(M_e / T_M) for e in [0, n_experts).
 * Picks the lexicographic minimum of (T(C), Delta_comp(C), C) over the legal C; rho is
 * quantised to 2^-20.  limits->force_comm_ctas > 0 wins over everything, then selector_off.
 * With limits->drain_help and rho->comm_warps_per_cta > 0 the candidate set is the product of C and the
 * number w of co-resident communication warps per compute CTA (w = 0 with C in 1..C_max, w in
 * 1..co_warps_max with C in 1..min(C_max, C_co_max)), T(C, w) follows the bandwidth-coupled recurrence
 * described at moe_rho, and the winner is the lexicographic minimum of (T, Delta_comp, w, C).
 * With drain_help = 0 and limits->dep_model = MOE_DEP_TILE the readiness of Eq. 9 is evaluated per
 * communication tile (from the routed tile counts: the last non-empty expert's tiles gate the tokens in
 * order) instead of per split.
 * Errors: MOE_ERR_PLAN_INFEASIBLE when no C (or the forced C) leaves P >= 1. */
int32_t plan_partition(const int32_t *routed_tile_counts, int32_t n_experts,
                       const moe_occupancy *occ, const moe_sm_limits *limits,
                       const moe_shape *shape, const moe_rho *rho, moe_plan *out);
/* The same selection when the routed counts exist only on the device (Section III-E): instead of
 * a device-to-host copy and a synchronisation made for scheduling alone, the counts are replaced
 * by a normalised-load estimate, R = T * k_tot assignments spread evenly over the E_tot experts:
 * ceil(ceil(R / E_tot) / tile_m) tiles each (the paper gives no formula; this is the reading taken).
 * out->W_comp then is the estimate, not the launch's tile count.  [host] */
int32_t plan_partition_estimate(const moe_occupancy *occ, const moe_sm_limits *limits,
                                const moe_shape *shape, const moe_rho *rho, moe_plan *out);

/* Mean cost [ns] of one plan_partition() call over `iters` calls rotating through n_sets
 * routed-count vectors (n_sets x n_experts ints, back to back).  The paper reports the
 * selector's standalone overhead (Section IV-B); this measures ours the same way.  [host] */
int32_t moe_time_plan_partition(const int32_t *routed_tile_counts, int32_t n_sets, int32_t n_experts,
                                const moe_occupancy *occ, const moe_sm_limits *limits,
                                const moe_shape *shape, const moe_rho *rho, int64_t iters,
                                double *mean_ns, int64_t *checksum);

/* ---- a3-a5: fused grouped GEMM2 + GatherRS combine --------------------------------------
 * Section II-A step 3, Section II-B (compute CTAs publish, communication CTAs consume),
 * Section III-C (CTA b takes global tiles b, b+P, ... of the split-major sequence; with
 * plan->drain_help the sequence is m-tile-major across the splits, so that x_routed is read once),
 * Section III-E (C* communication CTAs, R(C*) reserved SMs, P(C*) compute CTAs).
 *   out_d[t - d*ceil(T/EP)][:] = sum_j topk_w[t][j] * sum_p (x_routed[inv_perm[t,j]][Kp] . W2[e][:, Kp])
 * x_routed [device] bf16 [R, I]; W2 [device] bf16 [E_tot, H, I]; topk_w [device] fp32 [T, k_tot];
 * topk_idx is not read (the routing arrays already encode it) and may be NULL;
 * out [host] array of EP [device] pointers, buffer d is bf16 [ceil(T/EP), H], fully overwritten
 * for the tokens rank d owns; y_ws / flags_ws / status_dev as sized by moe_workspace_bytes.
 * n_mtiles = S (host value from moe_build_routing).  Requires H % 8 == 0, K % 16 == 0,
 * ceil(H/L) % 8 == 0, 16-byte aligned pointers, 1 <= C, 1 <= P, R * o_comm >= C,
 * R + ceil(P / o_comp) * comp_slot_sms <= G.
 * n_mtiles = MOE_MTILES_ON_DEVICE: the kernel reads S from the routing workspace itself (no host copy of
 * the counts is needed; the plan then comes from plan_partition_estimate). */
int32_t moe_gemm2_combine(moe_handle *h, const void *x_routed, const void *W2,
                          const int32_t *topk_idx, const float *topk_w,
                          const moe_shape *shape, const moe_occupancy *occ,
                          const moe_routing *routing, int32_t n_mtiles, const moe_plan *plan,
                          void *const *out, void *y_ws, uint32_t *flags_ws,
                          uint32_t *status_dev, void *stream);

/* The handle keeps, per flags workspace it has launched on, the launch epoch that marks a launch's readiness
 * flags (host memory: a small table keyed by the workspace address, touched by every moe_gemm2_combine; this is
 * why a handle serves one host thread at a time).  Call this before freeing a flags workspace, or before
 * zero-filling it again, so that the entry goes away and a later workspace at the same address starts from
 * epoch 0 with clean flags; flags_ws = NULL forgets every workspace.  A workspace must not be shared between
 * handles, and one that is reused without this call must not have been modified by anybody else.  [host] */
int32_t moe_release_workspace(moe_handle *h, const uint32_t *flags_ws);

/* Copies the 4-word device status to the host (synchronises the stream).  Returns
 * MOE_ERR_DEVICE_STATUS when code != 0. */
int32_t moe_get_status(moe_handle *h, const uint32_t *status_dev, moe_status *host, void *stream);
/* Clears the device status (asynchronous memset). */
int32_t moe_clear_status(moe_handle *h, uint32_t *status_dev, void *stream);

/* ---- the whole step on device-resident inputs -----------------------------------------------
 * One call for routing build -> wait for the tile counts -> plan_partition -> fused launch
 * (Section III-E: the manager sits between dispatch and launch; the counts are read on the host).
 * Inputs and workspaces as for moe_build_routing / moe_gemm2_combine; tile_counts_pinned [host]
 * E_tot + 1 ints, filled when the call returns; limits_or_null = NULL uses moe_query_occupancy's limits;
 * plan_out may be NULL.
 * Returns after the fused kernel has been launched (asynchronous on `stream`); the only host wait
 * inside is the one for the tile counts.  That wait is not a stream synchronisation: the routing kernel
 * that completes the counts stores them into the handle's pinned mailbox and then a sequence number;
 * the host polls that word (bounded: it gives up with MOE_ERR_CUDA when the stream finishes or fails
 * without the word, or after the handle's wait limit plus two seconds), copies the counts to
 * tile_counts_pinned, plans and launches while the routing build is still scattering, so that the
 * fused kernel is queued behind it without a gap (15 us per step on B200 against copy + synchronise).
 * If the mailbox could not be set up at moe_create the counts come by an asynchronous copy and a
 * stream synchronisation; tile_counts_pinned must then be pinned.  tile_counts_pinned = NULL selects the device-only-counts
 * path of Section III-E: no copy, no wait; the plan comes from plan_partition_estimate and the kernel
 * reads the tile count on the device (the whole call is then asynchronous; it is not meant for graph replay: the launch epoch that marks
 * this launch's flags is a kernel argument set by the host on every call).  ev_before / ev_after: optional cudaEvent_t handles (NULL = none)
 * recorded on `stream` right before and right after the fused launch, for timing it. */
int32_t moe_layer(moe_handle *h, const void *x_routed, const void *W2, const int32_t *topk_idx,
                  const float *topk_w, const moe_shape *shape, int32_t tile_m, int32_t tile_n,
                  const moe_sm_limits *limits_or_null, const moe_routing *routing,
                  int32_t *tile_counts_pinned, void *const *out, void *y_ws, uint32_t *flags_ws,
                  uint32_t *status_dev, moe_plan *plan_out, void *ev_before, void *ev_after, void *stream);

/* ---- the up-stream stage on the same GPU (Section II-A, steps 1-2; not changed by the paper) ------
 * x_routed[r][i] = silu(g) * u with g = hidden[t] . W1[e][0][i], u = hidden[t] . W1[e][1][i] for the routed
 * row r of assignment perm[r] = t * k_tot + j, e = topk_idx[t][j]; fp32 accumulation, bf16 result.  The
 * paper says "a gated activation" without naming it: SiLU gating is the reading taken.  Produces the
 * x_routed operand of moe_gemm2_combine in routed order.
 *   hidden      [device] bf16 [T, H], 16-byte aligned; H % 16 == 0, H >= 64
 *   W1          [device] bf16 [E_tot, 2, I, H] (plane 0 gate, plane 1 up; H contiguous); I % 16 == 0
 *   routing     a routing workspace built by moe_build_routing with this tile_m; n_mtiles as for
 *               moe_gemm2_combine (MOE_MTILES_ON_DEVICE allowed)
 *   h_routed_ws [device] moe_gemm1_workspace_bytes() bytes: the gathered rows [R, H]
 *   x_routed    [device] bf16 [R, I], 32-byte aligned, fully overwritten
 * Asynchronous on `stream` (one gather launch, one persistent tcgen05 launch); device-side problems go
 * to the status word like in moe_gemm2_combine. */
int32_t moe_gemm1_workspace_bytes(const moe_shape *shape, size_t *h_routed_bytes);
int32_t moe_gemm1_act(moe_handle *h, const void *hidden, const void *W1, const moe_shape *shape,
                      int32_t tile_m, const moe_routing *routing, int32_t n_mtiles, void *h_routed_ws,
                      void *x_routed, uint32_t *status_dev, void *stream);

/* ---- the post-router MoE layer on device-resident inputs (Section II-A: the three operations) ----
 * Routing build -> moe_gemm1_act (launched at once: it reads the m-tile count on the device) -> wait for
 * the tile counts (hidden behind GEMM1) -> plan_partition -> moe_gemm2_combine.  Arguments as for
 * moe_gemm1_act and moe_layer; x_routed_ws [device] bf16 [R, I], 32-byte aligned, is the intermediate.
 * tile_counts_pinned = NULL: no copy and no wait, plan from plan_partition_estimate.  A handle serves one
 * such call at a time (it owns the event the wait uses).  Asynchronous on `stream` after the wait. */
int32_t moe_post_router_layer(moe_handle *h, const void *hidden, const void *W1, const void *W2,
                              const int32_t *topk_idx, const float *topk_w, const moe_shape *shape,
                              int32_t tile_m, int32_t tile_n, const moe_sm_limits *limits_or_null,
                              const moe_routing *routing, int32_t *tile_counts_pinned, void *h_routed_ws,
                              void *x_routed_ws, void *const *out, void *y_ws, uint32_t *flags_ws,
                              uint32_t *status_dev, moe_plan *plan_out, void *stream);

/* ---- one-time service-rate characterisation of a kernel family (Eq. 13, Section III-C) -------
 * Measures rho_ref on the caller's reference workload (inputs and workspaces as for moe_layer): the
 * GEMM alone on P(C_ref) compute slots and the combine alone on C_ref communication CTAs (static
 * map), each n_samples (<= 64) launches after two warm-ups, median; rho_ref = time per communication
 * wave / time per compute wave.  Fills *rho_out with the constant and its reference factors (K, tile,
 * EP, rows per token, communication tile width; mode as moe_query_occupancy reports it), and
 * wave_us_out[0..1] (optional) with the two wave times in microseconds.  Meant to run once per kernel
 * family, never per workload; the stored constants of moe_query_occupancy were measured with it on
 * the DeepSeek-V2-Lite shape, T = 4096, uniform routing, TP = EP = L = 2, C_ref = 32.
 * Synchronises the stream; creates and destroys two CUDA events.  [host; device work on stream] */
int32_t moe_calibrate_rho(moe_handle *h, const void *x_routed, const void *W2, const int32_t *topk_idx,
                          const float *topk_w, const moe_shape *shape, int32_t tile_m, int32_t tile_n,
                          int32_t C_ref, int32_t n_samples, const moe_routing *routing,
                          int32_t *tile_counts_pinned, void *const *out, void *y_ws, uint32_t *flags_ws,
                          uint32_t *status_dev, moe_rho *rho_out, double *wave_us_out, void *stream);

/* ---- the whole step from host buffers ---------------------------------------------------
 * The call a user without device-resident activations makes: copies x_routed, topk_idx and
 * topk_w from (pinned) host memory into `arena`, builds the routing, waits for the tile
 * counts, plans, launches the fused kernel and copies the EP output blocks back to
 * out_host (bf16 [T, H], token order).  W2 stays device resident (weights).  Synchronous.
 * arena [device] of at least moe_host_arena_bytes(); plan_out may be NULL. */
int32_t moe_host_arena_bytes(const moe_shape *shape, int32_t tile_m, int32_t tile_n, size_t *bytes);
int32_t moe_layer_host(moe_handle *h, const void *x_routed_host, const int32_t *topk_idx_host,
                       const float *topk_w_host, const void *W2_dev, const moe_shape *shape,
                       int32_t tile_m, int32_t tile_n, const moe_sm_limits *limits_or_null,
                       void *arena, size_t arena_bytes, int32_t *tile_counts_pinned,
                       void *out_host, moe_plan *plan_out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H */
