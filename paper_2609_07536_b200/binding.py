"""ctypes binding of libmoe_b200.so: the same names as include/moe_b200.h, argument
marshalling only.  PyTorch supplies device memory (`tensor.data_ptr()`) and streams; every
step of the operator runs inside the library's CUDA kernels / host solver.

The library is mandatory: loading fails loudly when it has not been built
(`python -m paper_2609_07536_b200.build`); there is no fallback of any kind.
"""

from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libmoe_b200.so")

MOE_OK = 0
MOE_ERR_NULL, MOE_ERR_SHAPE, MOE_ERR_ALIGN, MOE_ERR_PLAN_INFEASIBLE = -1, -2, -3, -4
MOE_ERR_CUDA, MOE_ERR_UNSUPPORTED, MOE_ERR_DEVICE_STATUS, MOE_ERR_ARENA = -5, -6, -7, -8
MOE_ERR_STATIC_LIMIT = -9
MOE_DEV_OK, MOE_DEV_TIMEOUT, MOE_DEV_OOB, MOE_DEV_DUP_EXPERT = 0, 1, 2, 3
MOE_MODE_FUSED, MOE_MODE_GEMM_ONLY, MOE_MODE_COMBINE_ONLY = 0, 1, 2
MOE_RHO_PAPER, MOE_RHO_LOCAL = 0, 1
MOE_DEP_SPLIT, MOE_DEP_TILE = 0, 1
MOE_MAX_EP, MOE_MAX_L = 8, 8
MOE_MTILES_ON_DEVICE = -1

EXPORTS = [
    "moe_create", "moe_destroy", "moe_last_cuda_error", "moe_set_wait_limit_ns",
    "moe_query_occupancy", "moe_workspace_bytes", "moe_routing_view", "moe_build_routing",
    "moe_build_routing_static",
    "plan_partition", "plan_partition_estimate", "moe_time_plan_partition", "moe_gemm2_combine", "moe_get_status",
    "moe_clear_status",
    "moe_layer", "moe_calibrate_rho", "moe_host_arena_bytes", "moe_layer_host",
    "moe_gemm1_workspace_bytes", "moe_gemm1_act", "moe_post_router_layer", "moe_set_timeline",
    "moe_select_tile", "moe_release_workspace", "moe_set_probe",
]


class MoeError(RuntimeError):
    def __init__(self, code, what, detail=""):
        super().__init__(f"{what} failed with status {code}" + (f": {detail}" if detail else ""))
        self.code = code


class moe_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("T", "H", "I", "E_tot", "k_tot", "TP", "EP", "L")]


class moe_occupancy(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("tile_m", "tile_n", "comm_tile_m", "comm_tile_n", "o_comp", "o_comm",
                                                "comp_slot_sms")]


class moe_sm_limits(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("G", "C_max", "force_comm_ctas", "selector_off", "default_C",
                                                "drain_help", "co_warps_max", "force_co_warps", "C_co_max", "dep_model", "co_min_waves")]


class moe_rho(C.Structure):
    _fields_ = [("rho_ref", C.c_double)] + [(n, C.c_int32) for n in (
        "K_ref", "tile_m_ref", "tile_n_ref", "D_ref", "rows_ref", "comm_cols_ref", "mode",
        "comm_warps_per_cta", "n_sat_warps", "comm_quanta_per_tile", "reserved0")] + [("co_beta", C.c_double), ("co_gamma", C.c_double),
                                                 ("co_order", C.c_double)]


class moe_plan(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("comm_ctas", "R", "P", "W_comp", "W_comm", "delta")] + [
        ("pred_T_q", C.c_int64), ("rho_q", C.c_int64), ("mode", C.c_int32), ("debug_withhold_tile", C.c_int32),
        ("drain_help", C.c_int32), ("co_warps", C.c_int32)]


class moe_routing(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "counts", "offsets", "tiles", "tile_offsets", "perm", "inv_perm", "pad_row",
        "mtile_expert", "mtile_first_row", "mtile_valid", "scratch")] + [("max_mtiles", C.c_int32)]


class moe_status(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("code", "detail", "where", "count")]


TIMELINE_LIB_PATH = os.path.join(HERE, "libmoe_b200_timeline.so")
MOE_TIMELINE_SLOTS = 40

_lib = None
_lib_path = LIB_PATH


def use_timeline_library():
    """Selects the instrumented build (libmoe_b200_timeline.so) for this process; must come before the
    first call into the library."""
    global _lib_path
    if _lib is not None and _lib_path != TIMELINE_LIB_PATH:
        raise RuntimeError("the library is already loaded")
    _lib_path = TIMELINE_LIB_PATH


def lib():
    """The loaded library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_lib_path):
            raise ImportError(
                f"{_lib_path} is missing: build it with `python -m paper_2609_07536_b200.build"
                f"{' --timeline' if _lib_path == TIMELINE_LIB_PATH else ''}` (this package has no fallback path)")
        L = C.CDLL(_lib_path)
        vp, i32, u64 = C.c_void_p, C.c_int32, C.c_uint64
        P = C.POINTER
        L.moe_create.argtypes = [i32, P(vp)]
        L.moe_destroy.argtypes = [vp]
        L.moe_last_cuda_error.argtypes = [vp]
        L.moe_last_cuda_error.restype = C.c_char_p
        L.moe_set_wait_limit_ns.argtypes = [vp, u64]
        L.moe_query_occupancy.argtypes = [vp, i32, i32, P(moe_occupancy), P(moe_sm_limits), P(moe_rho)]
        L.moe_workspace_bytes.argtypes = [P(moe_shape), i32, i32] + [P(C.c_size_t)] * 4
        L.moe_routing_view.argtypes = [vp, P(moe_shape), i32, P(moe_routing)]
        L.moe_build_routing.argtypes = [vp, vp, P(moe_shape), i32, P(moe_routing), vp, vp, vp]
        L.moe_build_routing_static.argtypes = [vp, vp, P(moe_shape), i32, P(moe_routing), vp, vp, vp]
        L.plan_partition.argtypes = [P(i32), i32, P(moe_occupancy), P(moe_sm_limits), P(moe_shape),
                                     P(moe_rho), P(moe_plan)]
        L.plan_partition_estimate.argtypes = [P(moe_occupancy), P(moe_sm_limits), P(moe_shape), P(moe_rho),
                                              P(moe_plan)]
        L.moe_time_plan_partition.argtypes = [P(i32), i32, i32, P(moe_occupancy), P(moe_sm_limits),
                                              P(moe_shape), P(moe_rho), C.c_int64, P(C.c_double),
                                              P(C.c_int64)]
        L.moe_gemm2_combine.argtypes = [vp, vp, vp, vp, vp, P(moe_shape), P(moe_occupancy), P(moe_routing),
                                        i32, P(moe_plan), P(vp), vp, vp, vp, vp]
        L.moe_get_status.argtypes = [vp, vp, P(moe_status), vp]
        L.moe_clear_status.argtypes = [vp, vp, vp]
        L.moe_layer.argtypes = [vp, vp, vp, vp, vp, P(moe_shape), i32, i32, P(moe_sm_limits), P(moe_routing), vp,
                                P(vp), vp, vp, vp, P(moe_plan), vp, vp, vp]
        L.moe_calibrate_rho.argtypes = [vp, vp, vp, vp, vp, P(moe_shape), i32, i32, i32, i32, P(moe_routing), vp,
                                        P(vp), vp, vp, vp, P(moe_rho), P(C.c_double), vp]
        L.moe_gemm1_workspace_bytes.argtypes = [P(moe_shape), P(C.c_size_t)]
        L.moe_gemm1_act.argtypes = [vp, vp, vp, P(moe_shape), i32, P(moe_routing), i32, vp, vp, vp, vp]
        L.moe_post_router_layer.argtypes = [vp, vp, vp, vp, vp, vp, P(moe_shape), i32, i32, P(moe_sm_limits),
                                            P(moe_routing), vp, vp, vp, P(vp), vp, vp, vp, P(moe_plan), vp]
        L.moe_set_timeline.argtypes = [vp, vp, C.c_size_t]
        L.moe_select_tile.argtypes = [vp, P(moe_shape), P(i32), P(i32)]
        L.moe_release_workspace.argtypes = [vp, vp]
        L.moe_set_probe.argtypes = [vp, C.c_uint32]
        L.moe_host_arena_bytes.argtypes = [P(moe_shape), i32, i32, P(C.c_size_t)]
        L.moe_layer_host.argtypes = [vp, vp, vp, vp, vp, P(moe_shape), i32, i32, P(moe_sm_limits), vp,
                                     C.c_size_t, vp, vp, P(moe_plan), vp]
        for name in EXPORTS:
            if name != "moe_last_cuda_error":
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(rc, what, handle=None):
    if rc != MOE_OK:
        detail = ""
        if handle is not None and rc in (MOE_ERR_CUDA, MOE_ERR_STATIC_LIMIT, MOE_ERR_UNSUPPORTED):
            detail = (lib().moe_last_cuda_error(handle) or b"").decode()
        raise MoeError(rc, what, detail)


def _ptr(t):
    """Device / host address of a torch tensor, numpy array, int or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


# ----------------------------------------------------------------------------- the calls

def moe_create(device: int = 0):
    h = C.c_void_p()
    _check(lib().moe_create(device, C.byref(h)), "moe_create")
    return h


def moe_destroy(h):
    lib().moe_destroy(h)


def moe_set_wait_limit_ns(h, ns: int):
    _check(lib().moe_set_wait_limit_ns(h, ns), "moe_set_wait_limit_ns")


def moe_set_timeline(h, timeline_dev, nbytes: int):
    """Timeline build only: later fused launches record per-CTA stamps into `timeline_dev` (None: off)."""
    _check(lib().moe_set_timeline(h, _ptr(timeline_dev), nbytes), "moe_set_timeline", h)


def moe_select_tile(h, shape: moe_shape):
    """Kernel dispatch by shape: (tile_m, tile_n) of the GEMM tile family the library would use."""
    tm, tn = C.c_int32(), C.c_int32()
    _check(lib().moe_select_tile(h, C.byref(shape), C.byref(tm), C.byref(tn)), "moe_select_tile", h)
    return tm.value, tn.value


def moe_set_probe(h, probe_bits: int):
    """Timeline build only: leave out part of the data movement of later fused launches (garbage results)."""
    _check(lib().moe_set_probe(h, probe_bits), "moe_set_probe", h)


def moe_query_occupancy(h, tile_m: int, tile_n: int):
    occ, lim, rho = moe_occupancy(), moe_sm_limits(), moe_rho()
    _check(lib().moe_query_occupancy(h, tile_m, tile_n, C.byref(occ), C.byref(lim), C.byref(rho)),
           "moe_query_occupancy", h)
    return occ, lim, rho


def moe_workspace_bytes(shape: moe_shape, tile_m: int, tile_n: int):
    a, b, c, d = C.c_size_t(), C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(lib().moe_workspace_bytes(C.byref(shape), tile_m, tile_n, C.byref(a), C.byref(b), C.byref(c),
                                     C.byref(d)), "moe_workspace_bytes")
    return a.value, b.value, c.value, d.value


def moe_routing_view(routing_ws, shape: moe_shape, tile_m: int) -> moe_routing:
    r = moe_routing()
    _check(lib().moe_routing_view(_ptr(routing_ws), C.byref(shape), tile_m, C.byref(r)), "moe_routing_view")
    return r


def moe_build_routing(h, topk_idx, shape, tile_m, routing, tile_counts_host, status_dev, stream=None):
    _check(lib().moe_build_routing(h, _ptr(topk_idx), C.byref(shape), tile_m, C.byref(routing),
                                   _ptr(tile_counts_host), _ptr(status_dev), _stream(stream)),
           "moe_build_routing", h)


def moe_build_routing_static(h, topk_idx, shape, tile_m, routing, tile_counts_host, status_dev, stream=None):
    """Routing build whose scratch is a fixed array inside the library: for callers that cannot
    allocate device memory (frozen memory pools, allocator-owning frameworks, latency-critical
    sections).  Same results as moe_build_routing; `routing.scratch` is ignored.  Raises MoeError
    with code MOE_ERR_STATIC_LIMIT when ceil(T*k_tot/256) * E_tot exceeds 131072.  The first call
    on a device does a one-time set-up and should come before any stream capture; calls that
    overlap on the GPU race on the shared array."""
    _check(lib().moe_build_routing_static(h, _ptr(topk_idx), C.byref(shape), tile_m, C.byref(routing),
                                          _ptr(tile_counts_host), _ptr(status_dev), _stream(stream)),
           "moe_build_routing_static", h)


def plan_partition(routed_tile_counts, occ, limits, shape, rho) -> moe_plan:
    """routed_tile_counts: host int32 sequence of ceil(M_e / T_M)."""
    n = len(routed_tile_counts)
    arr = (C.c_int32 * n)(*[int(v) for v in routed_tile_counts])
    plan = moe_plan()
    _check(lib().plan_partition(arr, n, C.byref(occ), C.byref(limits), C.byref(shape), C.byref(rho),
                                C.byref(plan)), "plan_partition")
    return plan


def plan_partition_estimate(occ, limits, shape, rho) -> moe_plan:
    """The selection on the normalised-load estimate (routed counts left on the device)."""
    plan = moe_plan()
    _check(lib().plan_partition_estimate(C.byref(occ), C.byref(limits), C.byref(shape), C.byref(rho), C.byref(plan)),
           "plan_partition_estimate")
    return plan


def moe_time_plan_partition(count_sets, occ, limits, shape, rho, iters: int) -> float:
    """count_sets: list of equally long routed-count vectors.  Returns mean ns per call."""
    n_sets, n = len(count_sets), len(count_sets[0])
    flat = [int(v) for s in count_sets for v in s]
    arr = (C.c_int32 * len(flat))(*flat)
    mean, chk = C.c_double(), C.c_int64()
    _check(lib().moe_time_plan_partition(arr, n_sets, n, C.byref(occ), C.byref(limits), C.byref(shape),
                                         C.byref(rho), iters, C.byref(mean), C.byref(chk)),
           "moe_time_plan_partition")
    return mean.value


def moe_gemm2_combine(h, x_routed, W2, topk_idx, topk_w, shape, occ, routing, n_mtiles, plan, out,
                      y_ws, flags_ws, status_dev, stream=None):
    """out: sequence of EP device tensors, buffer d = bf16 [ceil(T/EP), H]."""
    outs = (C.c_void_p * len(out))(*[_ptr(o) for o in out])
    _check(lib().moe_gemm2_combine(h, _ptr(x_routed), _ptr(W2), _ptr(topk_idx), _ptr(topk_w),
                                   C.byref(shape), C.byref(occ), C.byref(routing), n_mtiles, C.byref(plan),
                                   outs, _ptr(y_ws), _ptr(flags_ws), _ptr(status_dev), _stream(stream)),
           "moe_gemm2_combine", h)


def moe_get_status(h, status_dev, stream=None, check: bool = True) -> moe_status:
    st = moe_status()
    rc = lib().moe_get_status(h, _ptr(status_dev), C.byref(st), _stream(stream))
    if rc not in (MOE_OK, MOE_ERR_DEVICE_STATUS) or (check and rc != MOE_OK):
        raise MoeError(rc, "moe_get_status",
                       f"device status code={st.code} detail={st.detail} where={st.where} count={st.count}")
    return st


def moe_release_workspace(h, flags_ws=None):
    """Forgets the launch epoch kept for `flags_ws` (None: for every workspace): call before freeing or
    re-zeroing a flags workspace."""
    _check(lib().moe_release_workspace(h, _ptr(flags_ws)), "moe_release_workspace", h)


def moe_clear_status(h, status_dev, stream=None):
    _check(lib().moe_clear_status(h, _ptr(status_dev), _stream(stream)), "moe_clear_status", h)


class LayerCall:
    """moe_layer with its arguments marshalled once (for a loop that repeats the same call)."""

    def __init__(self, h, x_routed, W2, topk_idx, topk_w, ws: "Workspace", limits=None, stream=None,
                 counts_on_device=False):
        self._stream = _stream(stream)
        self.h, self.ws = h, ws
        self.outs = (C.c_void_p * len(ws.out))(*[_ptr(o) for o in ws.out])
        self.plan = moe_plan()
        self.limits = limits
        self.args = (h, _ptr(x_routed), _ptr(W2), _ptr(topk_idx), _ptr(topk_w), C.byref(ws.shape), ws.tile_m,
                     ws.tile_n, C.byref(limits) if limits is not None else None, C.byref(ws.routing),
                     None if counts_on_device else _ptr(ws.tile_counts), self.outs, _ptr(ws.y_ws),
                     _ptr(ws.flags_ws), _ptr(ws.status),
                     C.byref(self.plan))
        self.keep = (x_routed, W2, topk_idx, topk_w)

    def __call__(self, ev_before=None, ev_after=None) -> moe_plan:
        """ev_before / ev_after: torch.cuda.Event objects that have been recorded at least once (so that
        their CUDA handles exist); they are re-recorded around the fused launch."""
        eb = ev_before.cuda_event if ev_before is not None else None
        ea = ev_after.cuda_event if ev_after is not None else None
        _check(lib().moe_layer(*self.args, eb, ea, self._stream), "moe_layer", self.h)
        return self.plan


def moe_layer(h, x_routed, W2, topk_idx, topk_w, ws: "Workspace", limits=None, stream=None,
              counts_on_device=False) -> moe_plan:
    """Routing build -> tile counts to the host -> analytical plan -> fused launch, in one library call.
    counts_on_device: no copy and no wait; the plan comes from the normalised-load estimate."""
    return LayerCall(h, x_routed, W2, topk_idx, topk_w, ws, limits, stream, counts_on_device)()


def moe_calibrate_rho(h, x_routed, W2, topk_idx, topk_w, ws: "Workspace", C_ref: int = 32, n_samples: int = 15,
                      stream=None):
    """One-time service-rate characterisation (Eq. 13) on the workload in `ws`.  Returns (moe_rho,
    us per compute wave, us per communication wave)."""
    outs = (C.c_void_p * len(ws.out))(*[_ptr(o) for o in ws.out])
    rho = moe_rho()
    waves = (C.c_double * 2)()
    _check(lib().moe_calibrate_rho(h, _ptr(x_routed), _ptr(W2), _ptr(topk_idx), _ptr(topk_w), C.byref(ws.shape),
                                   ws.tile_m, ws.tile_n, C_ref, n_samples, C.byref(ws.routing),
                                   _ptr(ws.tile_counts), outs, _ptr(ws.y_ws), _ptr(ws.flags_ws), _ptr(ws.status),
                                   C.byref(rho), waves, _stream(stream)), "moe_calibrate_rho", h)
    return rho, waves[0], waves[1]


def moe_gemm1_workspace_bytes(shape) -> int:
    b = C.c_size_t()
    _check(lib().moe_gemm1_workspace_bytes(C.byref(shape), C.byref(b)), "moe_gemm1_workspace_bytes")
    return b.value


def moe_gemm1_act(h, hidden, W1, shape, tile_m, routing, n_mtiles, h_routed_ws, x_routed, status_dev, stream=None):
    """Gather + grouped GEMM1 (gate, up) + silu(gate) * up -> x_routed [R, I] in routed order."""
    _check(lib().moe_gemm1_act(h, _ptr(hidden), _ptr(W1), C.byref(shape), tile_m, C.byref(routing), n_mtiles,
                               _ptr(h_routed_ws), _ptr(x_routed), _ptr(status_dev), _stream(stream)),
           "moe_gemm1_act", h)


def moe_post_router_layer(h, hidden, W1, W2, topk_idx, topk_w, ws: "Workspace", h_routed_ws, x_routed_ws,
                          limits=None, stream=None, counts_on_device=False) -> moe_plan:
    """Routing build -> GEMM1 + activation -> plan -> GEMM2 + combine, one library call."""
    outs = (C.c_void_p * len(ws.out))(*[_ptr(o) for o in ws.out])
    plan = moe_plan()
    _check(lib().moe_post_router_layer(h, _ptr(hidden), _ptr(W1), _ptr(W2), _ptr(topk_idx), _ptr(topk_w),
                                       C.byref(ws.shape), ws.tile_m, ws.tile_n,
                                       C.byref(limits) if limits is not None else None, C.byref(ws.routing),
                                       None if counts_on_device else _ptr(ws.tile_counts), _ptr(h_routed_ws),
                                       _ptr(x_routed_ws), outs, _ptr(ws.y_ws), _ptr(ws.flags_ws), _ptr(ws.status),
                                       C.byref(plan), _stream(stream)), "moe_post_router_layer", h)
    return plan


def moe_host_arena_bytes(shape, tile_m, tile_n) -> int:
    b = C.c_size_t()
    _check(lib().moe_host_arena_bytes(C.byref(shape), tile_m, tile_n, C.byref(b)), "moe_host_arena_bytes")
    return b.value


def moe_layer_host(h, x_routed_host, topk_idx_host, topk_w_host, W2_dev, shape, tile_m, tile_n, limits,
                   arena, arena_bytes, tile_counts_pinned, out_host, stream=None) -> moe_plan:
    plan = moe_plan()
    lim = C.byref(limits) if limits is not None else None
    _check(lib().moe_layer_host(h, _ptr(x_routed_host), _ptr(topk_idx_host), _ptr(topk_w_host), _ptr(W2_dev),
                                C.byref(shape), tile_m, tile_n, lim, _ptr(arena), arena_bytes,
                                _ptr(tile_counts_pinned), _ptr(out_host), C.byref(plan), _stream(stream)),
           "moe_layer_host", h)
    return plan


# ----------------------------------------------------------------------------- device memory plumbing

@dataclass
class Workspace:
    """Caller-owned buffers of one (shape, tile) configuration, allocated with torch."""
    shape: moe_shape
    tile_m: int
    tile_n: int
    routing_ws: object
    routing: moe_routing
    y_ws: object
    flags_ws: object
    status: object
    tile_counts: object     # pinned host int32 [E_tot + 1]
    out: list               # EP device tensors bf16 [ceil(T/EP), H]


def make_shape(T, H, I, E_tot, k_tot, TP, EP, L) -> moe_shape:
    return moe_shape(T, H, I, E_tot, k_tot, TP, EP, L)


def alloc_workspace(shape: moe_shape, tile_m: int, tile_n: int, device="cuda:0") -> Workspace:
    import torch
    rb, yb, fb, sb = moe_workspace_bytes(shape, tile_m, tile_n)
    routing_ws = torch.empty(rb, dtype=torch.uint8, device=device)
    y_ws = torch.empty(yb, dtype=torch.uint8, device=device)
    flags_ws = torch.zeros(fb, dtype=torch.uint8, device=device)      # zero-filled once
    status = torch.zeros(4, dtype=torch.int32, device=device)
    tile_counts = torch.zeros(shape.E_tot + 1, dtype=torch.int32).pin_memory()
    blk = -(-shape.T // shape.EP)
    out = [torch.empty((max(blk, 1), shape.H), dtype=torch.bfloat16, device=device) for _ in range(shape.EP)]
    routing = moe_routing_view(routing_ws, shape, tile_m)
    return Workspace(shape, tile_m, tile_n, routing_ws, routing, y_ws, flags_ws, status, tile_counts, out)
