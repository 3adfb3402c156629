"""Shared plumbing of the GPU parity tests: runs the library's path on a Workload through the
C-ABI binding and returns what the tests compare with the oracle."""

import numpy as np
import torch

from paper_2609_07536_b200 import binding as B
from paper_2609_07536_b200 import workloads as wl

_handle = None


def handle():
    global _handle
    if _handle is None:
        _handle = B.moe_create(0)
    return _handle


def shape_of(w: wl.Workload) -> B.moe_shape:
    return B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)


def routing_to_numpy(ws: B.Workspace, S: int) -> dict:
    """Copies the device routing arrays back (views into the routing workspace)."""
    s = ws.shape
    R, E = s.T * s.k_tot, s.E_tot
    base = ws.routing_ws.data_ptr()
    raw = ws.routing_ws.cpu().numpy()

    def view(ptr, n):
        off = ptr - base
        return raw[off:off + 4 * n].view(np.int32).copy()

    r = ws.routing
    return dict(counts=view(r.counts, E), offsets=view(r.offsets, E + 1), tiles=view(r.tiles, E),
                tile_offsets=view(r.tile_offsets, E + 1), perm=view(r.perm, R), inv_perm=view(r.inv_perm, R),
                pad_row=view(r.pad_row, R), mtile_expert=view(r.mtile_expert, S),
                mtile_first_row=view(r.mtile_first_row, S), mtile_valid=view(r.mtile_valid, S), S=S)


def build_routing(w: wl.Workload, topk_idx: np.ndarray, ws: B.Workspace = None):
    h = handle()
    shape = shape_of(w)
    if ws is None:
        ws = B.alloc_workspace(shape, w.tile_m, w.tile_n)
    idx_dev = torch.from_numpy(np.ascontiguousarray(topk_idx)).cuda() if topk_idx.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    B.moe_clear_status(h, ws.status)
    B.moe_build_routing(h, idx_dev, shape, w.tile_m, ws.routing, ws.tile_counts, ws.status)
    torch.cuda.synchronize()
    S = int(ws.tile_counts[shape.E_tot])
    return ws, idx_dev, S


def run_layer(w: wl.Workload, topk_idx, topk_w, x, W2, force_C=0, mode=B.MOE_MODE_FUSED, ws=None,
              withhold=-1, check_status=True, P_override=None, drain_help=None, co_warps=0, C_override=None):
    """x, W2: bf16 torch tensors (CPU or CUDA).  Returns (list of EP outputs on CPU as float32,
    plan, workspace, S)."""
    h = handle()
    shape = shape_of(w)
    ws, idx_dev, S = build_routing(w, topk_idx, ws)
    occ, lim, rho = B.moe_query_occupancy(h, w.tile_m, w.tile_n)
    lim.force_comm_ctas = force_C
    if drain_help is not None:
        lim.drain_help = int(drain_help)
    lim.force_co_warps = int(co_warps)
    tiles = ws.tile_counts[:shape.E_tot].tolist()
    plan = B.plan_partition(tiles, occ, lim, shape, rho)
    plan.mode = mode
    plan.debug_withhold_tile = withhold
    if P_override is not None:
        plan.P = P_override
    if C_override is not None:
        plan.comm_ctas = plan.R = C_override
    xd, Wd = x.cuda(), W2.cuda()
    wd = torch.from_numpy(np.ascontiguousarray(topk_w)).cuda() if topk_w.size else torch.zeros(1, device="cuda")
    for o in ws.out:
        o.fill_(float("nan"))
    B.moe_gemm2_combine(h, xd, Wd, idx_dev, wd, shape, occ, ws.routing, S, plan, ws.out, ws.y_ws,
                        ws.flags_ws, ws.status)
    torch.cuda.synchronize()
    st = B.moe_get_status(h, ws.status, check=check_status)
    outs = [o.float().cpu().numpy() for o in ws.out]
    return outs, plan, ws, S, st


def tokens_of_rank(T, EP, d):
    blk = -(-T // EP)
    return range(min(T, d * blk), min(T, (d + 1) * blk))


def tolerance(ref: np.ndarray) -> float:
    """max |err| <= 1e-2 * rms(ref) + 1e-3 (bf16 in, fp32 accumulate)."""
    rms = float(np.sqrt(np.mean(np.square(ref.astype(np.float64))))) if ref.size else 0.0
    return 1e-2 * rms + 1e-3
