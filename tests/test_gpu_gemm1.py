"""GPU parity of the up-stream stage (gather + grouped GEMM1 + gated activation) against the CPU
oracle, through the C ABI."""

from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import gemm1_act_ref as g1
from oracle import gemm2_combine_ref as g2
from oracle import routing_ref as rr
from paper_2609_07536_b200 import binding as B
from paper_2609_07536_b200 import workloads as wl
from tests import gpu_common as G

pytestmark = pytest.mark.gpu


def _run(w, idx, hidden, W1, counts_on_device=False):
    h = G.handle()
    ws, idx_d, S = G.build_routing(w, idx, None)
    shape = ws.shape
    hr = torch.empty(B.moe_gemm1_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    x = torch.full((w.R, w.I), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.moe_gemm1_act(h, hidden.cuda(), W1.cuda(), shape, w.tile_m, ws.routing,
                    B.MOE_MTILES_ON_DEVICE if counts_on_device else S, hr, x, ws.status)
    torch.cuda.synchronize()
    assert B.moe_get_status(h, ws.status).code == 0
    return x, ws


def _tolerance(ref):
    # bf16 output: its own rounding (2^-9 relative, 2^-8 allowed) on top of the path's tolerance
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2))) if ref.size else 0.0
    return 1e-2 * rms + 1e-3 + 2.0 ** -8 * np.abs(ref)


def _check(w, n_rows=None, **kw):
    idx, _, _ = wl.make_routing(w)
    hidden, W1 = wl.make_gemm1_data(w)
    x, ws = _run(w, idx, hidden, W1, **kw)
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    if n_rows is None or n_rows >= w.R:
        rows = np.arange(w.R, dtype=np.int32)
    else:
        rng = np.random.default_rng(1)
        pick = set(rng.choice(w.R, size=n_rows, replace=False).tolist())
        for e in range(w.E_tot):                       # first and last row of every expert, rows of partial m-tiles
            lo, hi = int(r["offsets"][e]), int(r["offsets"][e + 1])
            if hi > lo:
                pick.update({lo, hi - 1, lo + (hi - lo - 1) // 128 * 128})
        rows = np.array(sorted(pick), dtype=np.int32)
    ref = g1.gemm1_act(wl.bf16_bits(hidden), wl.bf16_bits(W1), idx, r["perm"], rows=rows)
    got = x.float().cpu().numpy()[rows]
    assert not np.isnan(got).any()
    assert np.all(np.abs(got - ref) <= _tolerance(ref)), float(np.max(np.abs(got - ref)))
    return x, ws, idx, r


def test_tiny_all_rows():
    _check(wl.TINY)


@pytest.mark.parametrize("kw", [
    dict(T=1, E=4, k=2, H=64, I=16, tile_m=64),                       # one token, a 16-column tile
    dict(T=333, E=12, k=3, H=272, I=208, tile_m=64, EP=1),            # ragged rows, partial k-block and n-tile
    dict(T=1030, E=70, k=2, H=512, I=384, tile_m=128),                # empty experts
    dict(T=700, E=6, k=2, n_shared=2, H=256, I=128, tile_m=256, tile_n=256),  # shared experts, 256-row m-tiles
], ids=lambda kw: "-".join(f"{k}{v}" for k, v in kw.items()))
def test_edge_shapes(kw):
    base = dict(name="g1edge", routing_seed=7, data_seed=8, TP=1, EP=1, L=1, tile_n=64)
    base.update(kw)
    _check(replace(wl.TINY, **base))


def test_granite_and_dsv2lite_shapes_sampled():
    _check(wl.GRANITE, n_rows=300)
    _check(wl.DSV2L, n_rows=200, counts_on_device=True)


def test_same_bits_for_every_m_tile_size():
    # the m-tile size only changes which CTA computes a row, never the arithmetic of the row
    w = replace(wl.GRANITE, name="g1bits", T=900)
    idx, _, _ = wl.make_routing(w)
    hidden, W1 = wl.make_gemm1_data(w)
    base = None
    for tm in (64, 128, 256):
        x, _ = _run(replace(w, tile_m=tm), idx, hidden, W1)
        bits = x.view(torch.int16).cpu().numpy()
        if base is None:
            base = bits
        assert np.array_equal(base, bits), tm


def test_output_feeds_the_down_projection():
    # GEMM1's x_routed goes straight into GEMM2 + combine; the layer's output matches the oracle's GEMM2
    # evaluated on the very bits GEMM1 produced
    w = replace(wl.TINY, name="chain", T=300, E=6, k=2, H=128, I=128, TP=1, EP=2, tile_m=128, tile_n=128)
    idx, wt, _ = wl.make_routing(w)
    hidden, W1 = wl.make_gemm1_data(w)
    _, W2 = wl.make_data(w)
    x, ws = _run(w, idx, hidden, W1)
    outs, plan, ws2, S, st = G.run_layer(w, idx, wt, x, W2, ws=ws)
    assert st.code == 0
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    expect = g2.gemm2_combine(wl.bf16_bits(x.cpu()), wl.bf16_bits(W2), idx, wt, r["inv_perm"])
    got = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(outs)])
    assert np.max(np.abs(got - expect)) <= G.tolerance(expect)


def test_argument_validation():
    h = G.handle()
    w = wl.TINY
    idx, _, _ = wl.make_routing(w)
    hidden, W1 = wl.make_gemm1_data(w)
    ws, idx_d, S = G.build_routing(w, idx, None)
    hr = torch.empty(B.moe_gemm1_workspace_bytes(ws.shape), dtype=torch.uint8, device="cuda")
    x = torch.empty((w.R, w.I), dtype=torch.bfloat16, device="cuda")
    hd, Wd = hidden.cuda(), W1.cuda()
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm1_act(h, hd, Wd, ws.shape, 96, ws.routing, S, hr, x, ws.status)
    assert e.value.code == B.MOE_ERR_UNSUPPORTED
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm1_act(h, hd, Wd, ws.shape, w.tile_m, ws.routing, S, hr, x.data_ptr() + 2, ws.status)
    assert e.value.code == B.MOE_ERR_ALIGN
    bad = B.make_shape(w.T, w.H, w.I + 8, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm1_act(h, hd, Wd, bad, w.tile_m, ws.routing, S, hr, x, ws.status)
    assert e.value.code == B.MOE_ERR_SHAPE


@pytest.mark.parametrize("counts_on_device", [False, True], ids=["host_counts", "device_counts"])
def test_post_router_layer_against_the_oracle_chain(counts_on_device):
    # the three operations of Section II-A in one call, against the oracle's GEMM1 + activation (rounded to
    # bf16 as the stored intermediate is) followed by the oracle's GEMM2 + combine
    h = G.handle()
    w = replace(wl.TINY, name="layer3", T=500, E=10, k=3, n_shared=1, H=256, I=256, TP=2, EP=2, L=2,
                tile_m=128, tile_n=128, routing="zipf", zipf_s=1.0, target_r_expert=2.0)
    idx, wt, _ = wl.make_routing(w)
    hidden, W1 = wl.make_gemm1_data(w)
    _, W2 = wl.make_data(w)
    ws = B.alloc_workspace(G.shape_of(w), w.tile_m, w.tile_n)
    hr = torch.empty(B.moe_gemm1_workspace_bytes(ws.shape), dtype=torch.uint8, device="cuda")
    xr = torch.empty((w.R, w.I), dtype=torch.bfloat16, device="cuda")
    idx_d, wt_d = torch.from_numpy(idx).cuda(), torch.from_numpy(wt).cuda()
    for o in ws.out:
        o.fill_(float("nan"))
    plan = B.moe_post_router_layer(h, hidden.cuda(), W1.cuda(), W2.cuda(), idx_d, wt_d, ws, hr, xr,
                                   counts_on_device=counts_on_device)
    torch.cuda.synchronize()
    assert B.moe_get_status(h, ws.status).code == 0 and plan.comm_ctas >= 1
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    x_ref = g1.gemm1_act(wl.bf16_bits(hidden), wl.bf16_bits(W1), idx, r["perm"])
    x_bits = wl.bf16_bits(torch.from_numpy(x_ref).bfloat16())
    expect = g2.gemm2_combine(x_bits, wl.bf16_bits(W2), idx, wt, r["inv_perm"])
    outs = [o.float().cpu().numpy() for o in ws.out]
    got = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(outs)])
    assert not np.isnan(got).any()
    # the intermediate may differ from the oracle's by one bf16 step in a few places: same tolerance form
    assert np.max(np.abs(got - expect)) <= G.tolerance(expect)


def test_random_small_shapes_against_the_oracle():
    # seeded fuzz: ragged token counts, partial k-blocks and n-tiles, every m-tile size, empty experts
    rng = np.random.default_rng(77)
    for case in range(14):
        tile_m = int(rng.choice([64, 128, 256]))
        w = replace(wl.TINY, name=f"g1fuzz{case}", T=int(rng.choice([1, 9, 130, 257, 600])),
                    H=int(rng.choice([64, 80, 144, 256, 528])), I=int(rng.choice([16, 48, 128, 144, 272])),
                    E=int(rng.integers(1, 24)), k=1, n_shared=int(rng.choice([0, 1])), TP=1, EP=1, L=1,
                    tile_m=tile_m, tile_n=256 if tile_m == 256 else 64, routing_seed=300 + case, data_seed=400 + case)
        w = replace(w, k=int(rng.integers(1, min(w.E, 3) + 1)))
        _check(w, counts_on_device=bool(rng.integers(2)))
