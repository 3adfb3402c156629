"""moe_build_routing_static: the routing build for callers that cannot allocate device memory
(serving loops with a frozen memory pool, frameworks that own the allocator, latency-critical
sections).  Its scratch is a fixed array inside the library, so this test checks, through the
C ABI, that it produces exactly what moe_build_routing produces with a caller-allocated
workspace and what the CPU routing reference computes -- twice in a row on different inputs,
because the shared array keeps the previous call's contents --, that the amount of free device
memory does not move across the calls, and that a problem too large for the array is refused
with a clear error.

Collected last on purpose (file name), and independent of the other tests: it builds its own
handle and workspaces, so it passes alone in a fresh process as well as after the others.
"""

from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import routing_ref as rr
from paper_2609_07536_b200 import binding as B
from paper_2609_07536_b200 import workloads as wl

pytestmark = pytest.mark.gpu

KEYS = ["counts", "offsets", "tiles", "tile_offsets", "perm", "inv_perm", "pad_row",
        "mtile_expert", "mtile_first_row", "mtile_valid"]


def _arrays(ws, S):
    s = ws.shape
    R, E = s.T * s.k_tot, s.E_tot
    base = ws.routing_ws.data_ptr()
    raw = ws.routing_ws.cpu().numpy()
    view = lambda ptr, n: raw[ptr - base:ptr - base + 4 * n].view(np.int32).copy()
    r = ws.routing
    sizes = dict(counts=E, offsets=E + 1, tiles=E + 1, tile_offsets=E + 1, perm=R, inv_perm=R, pad_row=R,
                 mtile_expert=S, mtile_first_row=S, mtile_valid=S)
    return {k: view(getattr(r, k), n) for k, n in sizes.items()}


def _run(h, fn, w, idx, null_scratch=False):
    shape = B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
    ws = B.alloc_workspace(shape, w.tile_m, w.tile_n)
    ws.routing_ws.fill_(0x5A)                       # stale bytes must not matter
    if null_scratch:
        ws.routing.scratch = None                   # the static variant never touches it
    idx_d = torch.from_numpy(idx).cuda()
    fn(h, idx_d, shape, w.tile_m, ws.routing, ws.tile_counts, ws.status)
    torch.cuda.synchronize()
    st = B.moe_get_status(h, ws.status)
    assert st.code == 0
    S = int(ws.tile_counts[w.E_tot])
    return _arrays(ws, S), ws.tile_counts.clone(), S


def test_static_scratch_variant_matches_the_workspace_variant_twice_in_a_row():
    h = B.moe_create(0)
    try:
        cases = [wl.DSV2L, replace(wl.GRANITE, T=1000, routing_seed=5), wl.TINY]
        for w in cases:                              # consecutive calls share the built-in array
            idx, _, _ = wl.make_routing(w)
            ref, ref_counts, S_ref = _run(h, B.moe_build_routing, w, idx)
            got, got_counts, S = _run(h, B.moe_build_routing_static, w, idx, null_scratch=True)
            assert S == S_ref and torch.equal(ref_counts, got_counts)
            want = rr.build_routing(idx, w.E_tot, w.tile_m)          # the CPU reference, directly
            assert S == want["S"]
            for k in KEYS:                           # integer work: bit-exact
                assert np.array_equal(ref[k], got[k]), (w.name, k)
                n = len(want[k])
                assert np.array_equal(got[k][:n], np.asarray(want[k], dtype=np.int32)), (w.name, k, "vs reference")
        # and the very same input twice
        idx, _, _ = wl.make_routing(wl.DSV2L)
        a, _, _ = _run(h, B.moe_build_routing_static, wl.DSV2L, idx, null_scratch=True)
        b, _, _ = _run(h, B.moe_build_routing_static, wl.DSV2L, idx, null_scratch=True)
        for k in KEYS:
            assert np.array_equal(a[k], b[k]), k
    finally:
        B.moe_destroy(h)


def test_later_calls_leave_the_amount_of_free_device_memory_alone():
    """The point of the entry point: nothing is allocated.  The first call may make the driver load
    the module that holds the array; from the second call on, free device memory as the driver
    reports it must not move (the test's own buffers are all allocated beforehand)."""
    h = B.moe_create(0)
    try:
        w = replace(wl.GRANITE, T=2048, routing_seed=9)
        idx, _, _ = wl.make_routing(w)
        shape = B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
        ws = B.alloc_workspace(shape, w.tile_m, w.tile_n)
        ws.routing.scratch = None
        idx_d = torch.from_numpy(idx).cuda()
        B.moe_build_routing_static(h, idx_d, shape, w.tile_m, ws.routing, ws.tile_counts, ws.status)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        reserved_before = torch.cuda.memory_reserved()
        for _ in range(3):
            B.moe_build_routing_static(h, idx_d, shape, w.tile_m, ws.routing, ws.tile_counts, ws.status)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert torch.cuda.memory_reserved() == reserved_before      # nothing went through torch's allocator
        assert free_after == free_before, (free_before, free_after)  # nor through cudaMalloc
        assert B.moe_get_status(h, ws.status).code == 0
    finally:
        B.moe_destroy(h)


def test_sizes_beyond_the_builtin_array_are_refused():
    h = B.moe_create(0)
    try:
        # ceil(65536 * 8 / 256) * 66 = 135168 > 131072
        w = replace(wl.DSV2L, T=65536)
        shape = B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
        rb, _, _, _ = B.moe_workspace_bytes(shape, w.tile_m, w.tile_n)
        routing_ws = torch.empty(rb, dtype=torch.uint8, device="cuda")
        routing = B.moe_routing_view(routing_ws, shape, w.tile_m)
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        idx_d = torch.zeros((w.T, w.k_tot), dtype=torch.int32, device="cuda")
        with pytest.raises(B.MoeError) as e:
            B.moe_build_routing_static(h, idx_d, shape, w.tile_m, routing, None, status)
        assert e.value.code == B.MOE_ERR_STATIC_LIMIT
        assert "131072" in str(e.value) and "moe_build_routing" in str(e.value)
        torch.cuda.synchronize()
        assert int(status[0]) == 0                   # nothing was launched
    finally:
        B.moe_destroy(h)
