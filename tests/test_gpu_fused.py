"""Fused GEMM2 + combine (CUDA, through the C ABI) against the CPU oracle.

Tolerance (bf16 inputs, fp32 accumulation, bf16 intermediate and output):
    max |err| <= 1e-2 * rms(ref) + 1e-3
Integer work (routing) is compared bit-exactly in test_gpu_routing.py.  Where several results
are correct (summation order) the tolerance applies; what must be unique is checked as such:
the GPU result is bitwise identical for every C, every P and from run to run.
"""

from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import gemm2_combine_ref as ref
from oracle import routing_ref as rr
from paper_2609_07536_b200 import binding as B
from paper_2609_07536_b200 import workloads as wl
from tests import gpu_common as G

pytestmark = pytest.mark.gpu


def _oracle_tokens(w, idx, wt, x, W2, tokens=None):
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    return ref.gemm2_combine(wl.bf16_bits(x), wl.bf16_bits(W2), idx, wt, r["inv_perm"], tokens=tokens), r


def _gather_tokens(outs, T, EP, tokens):
    blk = -(-T // EP)
    return np.stack([outs[t // blk][t % blk] for t in tokens])


def _stratified_tokens(w, idx, r, n_random, seed=0):
    """first/last tokens of each rank block, tokens sitting in partial m-tiles, tokens of the
    hottest and the coldest expert, and a random rest."""
    rng = np.random.default_rng(seed)
    T, k_tot = idx.shape
    blk = -(-T // w.EP)
    toks = set()
    for d in range(w.EP):
        lo, hi = min(T, d * blk), min(T, (d + 1) * blk)
        toks.update(range(lo, min(hi, lo + 3)))
        toks.update(range(max(lo, hi - 3), hi))
    partial = np.nonzero(r["mtile_valid"] < w.tile_m)[0][:8]
    for mu in partial:
        row = r["mtile_first_row"][mu] + r["mtile_valid"][mu] - 1
        toks.add(int(r["perm"][row]) // k_tot)
    counts = r["counts"].copy()
    hot = int(np.argmax(counts))
    cold = int(np.argmin(np.where(counts > 0, counts, counts.max() + 1)))
    for e in (hot, cold):
        rows = range(r["offsets"][e], min(r["offsets"][e + 1], r["offsets"][e] + 4))
        toks.update(int(r["perm"][row]) // k_tot for row in rows)
    toks.update(int(t) for t in rng.choice(T, size=min(T, n_random), replace=False))
    return np.array(sorted(toks), dtype=np.int32)


def _check_against_oracle(w, n_random=None, **run_kw):
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2, **run_kw)
    assert st.code == 0
    if n_random is None:
        expect, r = _oracle_tokens(w, idx, wt, x, W2)
        tokens = np.arange(w.T)
    else:
        r = rr.build_routing(idx, w.E_tot, w.tile_m)
        tokens = _stratified_tokens(w, idx, r, n_random)
        expect, _ = _oracle_tokens(w, idx, wt, x, W2, tokens=tokens)
    got = _gather_tokens(outs, w.T, w.EP, tokens) if len(tokens) else np.zeros((0, w.H), np.float32)
    assert not np.isnan(got).any()
    tol = G.tolerance(expect)
    err = float(np.max(np.abs(got - expect))) if got.size else 0.0
    assert err <= tol, (w.name, err, tol)
    # nothing but the owned rows is written: untouched tail rows of a short last block stay NaN
    return outs, plan


def test_tiny_config_all_tokens():
    outs, plan = _check_against_oracle(wl.TINY)
    assert plan.comm_ctas >= 1 and plan.P >= 1


def test_granite_config_all_tokens():
    _check_against_oracle(wl.GRANITE)


def test_qwen_config_sampled():
    _check_against_oracle(wl.QWEN, n_random=384)


def test_dsv2lite_config_sampled_in_bench_configuration():
    # the launch configuration bench.py times: analytical plan, 256x256 CTA-pair tiles, L = 2
    _check_against_oracle(wl.DSV2L, n_random=160)


@pytest.mark.parametrize("kw", [
    dict(T=1, E=4, k=2, H=64, I=64, tile_m=64, tile_n=64),                 # a single token
    dict(T=333, E=12, k=3, H=264, I=80, tile_m=64, tile_n=64, EP=4),       # ragged everything; K = 80
    dict(T=777, E=5, k=2, H=1536, I=512, TP=2, EP=3, tile_m=128, tile_n=256, L=4),  # split 384: partial n-tile
    dict(T=513, E=3, k=1, H=2048, I=352 * 4, TP=4, EP=2, tile_m=128, tile_n=128, L=2),  # K = 352: partial k-block
    dict(T=1030, E=70, k=2, H=512, I=256, TP=2, EP=8, tile_m=128, tile_n=128, L=8),  # empty experts, L = 8
    dict(T=200, E=6, k=2, n_shared=2, H=256, I=128, TP=1, EP=1, tile_m=128, tile_n=64, L=2),  # shared experts
], ids=lambda kw: "-".join(f"{k}{v}" for k, v in kw.items()))
@pytest.mark.parametrize("drain_help", [0, 1], ids=["static", "drain_help"])
def test_edge_shapes(kw, drain_help):
    # both ways of handing out the communication work: the paper's static tile -> CTA map, and warps
    # pulling token ranges from the two-ended queue (for a forced C that leaves most of it to helpers)
    base = dict(name="edge", routing_seed=3, data_seed=4, TP=1, EP=1, L=1)
    base.update(kw)
    w = replace(wl.TINY, **base)
    _check_against_oracle(w, drain_help=drain_help)
    _check_against_oracle(w, drain_help=drain_help, force_C=2)


def test_one_hot_expert_and_forced_counts():
    w = replace(wl.TINY, name="hot", T=900, E=8, k=1, H=512, I=256, TP=2, EP=2, tile_m=128, tile_n=256)
    idx = np.full((w.T, 1), 5, dtype=np.int32)
    wt = np.ones((w.T, 1), dtype=np.float32)
    x, W2 = wl.make_data(w)
    expect, _ = _oracle_tokens(w, idx, wt, x, W2)
    for C in (1, 3, 40, 147):
        outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2, force_C=C)
        assert plan.comm_ctas == C and plan.P == 148 - C and st.code == 0
        got = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(outs)])
        assert np.max(np.abs(got - expect)) <= G.tolerance(expect)


def test_bitwise_identical_across_C_P_and_runs():
    w = replace(wl.GRANITE, name="det", T=1536)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    base = None
    for C, P in [(0, None), (1, None), (2, None), (7, None), (33, None), (74, None), (147, None), (5, 9), (5, 1)]:
        for rep in range(2):
            outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2, force_C=C, P_override=P)
            assert st.code == 0
            bits = [torch.from_numpy(o).bfloat16().view(torch.int16).numpy() for o in outs]
            if base is None:
                base = bits
            for a, b in zip(base, bits):
                assert np.array_equal(a, b), (C, P, rep)


def test_drain_help_and_tile_families_change_nothing_but_time():
    # compute CTAs helping with the communication tail, or another GEMM tile family, may only change
    # who writes a value and when: the bits must be the same
    w = replace(wl.GRANITE, name="dh", T=2000, L=2)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    base = None
    for tile in ((128, 256), (128, 128), (256, 256)):
        for dh in (0, 1):
            for C in (0, 1, 9, 60):
                wt_ = replace(w, tile_m=tile[0], tile_n=tile[1])
                outs, plan, ws, S, st = G.run_layer(wt_, idx, wt, x, W2, force_C=C, drain_help=dh)
                assert st.code == 0 and plan.drain_help == dh
                bits = [torch.from_numpy(o).bfloat16().view(torch.int16).numpy() for o in outs]
                if base is None:
                    base = bits
                for a, b in zip(base, bits):
                    assert np.array_equal(a, b), (tile, dh, C)
    expect, _ = _oracle_tokens(w, idx, wt, x, W2)
    got = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(outs)])
    assert np.max(np.abs(got - expect)) <= G.tolerance(expect)


def test_co_resident_communication_warps_change_nothing_but_time():
    # extra communication warps inside every compute CTA (they serve split s while the CTA computes split
    # s + 1), with or without dedicated communication CTAs, in both kernels: same bits as the plain launch,
    # and those bits are the oracle's result within the path's tolerance
    w = replace(wl.GRANITE, name="co", T=2000, L=2)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    base = None
    for tile in ((128, 256), (256, 256), (128, 128)):
        for co, C, C_override in ((0, 1, None), (1, 1, None), (2, 1, None), (2, 9, None), (2, 1, 0), (1, 1, 0)):
            wt_ = replace(w, tile_m=tile[0], tile_n=tile[1])
            P_override = (148 // (2 if tile[0] == 256 else 1)) if C_override == 0 else None
            outs, plan, ws, S, st = G.run_layer(wt_, idx, wt, x, W2, force_C=C, drain_help=1, co_warps=co,
                                                C_override=C_override, P_override=P_override)
            assert st.code == 0 and plan.co_warps == co
            bits = [torch.from_numpy(o).bfloat16().view(torch.int16).numpy() for o in outs]
            if base is None:
                base = bits
            for a, b in zip(base, bits):
                assert np.array_equal(a, b), (tile, co, C, C_override)
    expect, _ = _oracle_tokens(w, idx, wt, x, W2)
    got = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(outs)])
    assert np.max(np.abs(got - expect)) <= G.tolerance(expect)


@pytest.mark.parametrize("kw", [
    dict(T=777, E=5, k=2, H=1536, I=512, TP=2, EP=3, tile_m=128, tile_n=256, L=4),   # partial n-tile at the split end
    dict(T=1030, E=70, k=2, H=512, I=256, TP=2, EP=8, tile_m=128, tile_n=128, L=8),  # empty experts, L = 8
    dict(T=200, E=6, k=2, n_shared=2, H=256, I=128, TP=1, EP=1, tile_m=128, tile_n=64, L=2),  # shared experts
    dict(T=900, E=9, k=4, H=1024, I=256, TP=4, EP=2, tile_m=256, tile_n=256, L=2),    # pair tiles, 16-row units
    dict(T=333, E=12, k=3, H=264, I=80, tile_m=64, tile_n=64, EP=4, L=1),             # no room for them: dropped
], ids=lambda kw: "-".join(f"{k}{v}" for k, v in kw.items()))
def test_co_resident_warps_edge_shapes(kw):
    base = dict(name="co_edge", routing_seed=5, data_seed=6, TP=1, EP=1, L=1)
    base.update(kw)
    w = replace(wl.TINY, **base)
    _check_against_oracle(w, drain_help=1, co_warps=2)
    _check_against_oracle(w, drain_help=1, co_warps=1, force_C=3)


def test_dsv2lite_with_co_resident_warps_sampled():
    _check_against_oracle(wl.DSV2L, n_random=96, co_warps=2)


@pytest.mark.parametrize("T", [16, 64, 256, 1024])
def test_decode_sized_token_counts_on_the_deepseek_shape(T):
    # small and decode-sized batches (every expert holds a handful of rows): the tile family comes from the
    # library's dispatch by shape, every token is checked
    w = replace(wl.DSV2L, name=f"decode{T}", T=T)
    tm, tn = B.moe_select_tile(G.handle(), G.shape_of(w))
    assert (tm, tn) == (128, 256)
    _check_against_oracle(replace(w, tile_m=tm, tile_n=tn))


def test_dispatch_by_shape():
    h = G.handle()
    sel = lambda w: B.moe_select_tile(h, G.shape_of(w))
    assert sel(wl.DSV2L) == (256, 256) and sel(replace(wl.DSV2L, T=2048)) == (256, 256)    # >= 192 routed rows per expert
    assert sel(wl.QWEN) == (256, 256) and sel(wl.GRANITE) == (256, 256)                    # 546 and 819 rows per expert
    assert sel(replace(wl.DSV2L, T=1024)) == (128, 256) and sel(replace(wl.DSV2L, T=1)) == (128, 256)   # 124 rows and fewer
    assert sel(replace(wl.DSV2L, L=8)) == (256, 256)                            # split width 256
    assert sel(replace(wl.DSV2L, L=4, H=512)) == (128, 128)                     # split width 128: no pair tile
    assert sel(wl.TINY) == (128, 256) and sel(replace(wl.TINY, H=64)) == (128, 64)
    with pytest.raises(B.MoeError):
        sel(replace(wl.TINY, H=250))
    # whatever it returns is a configuration the other calls accept
    for w in (wl.DSV2L, wl.GRANITE, replace(wl.TINY, H=64)):
        tm, tn = sel(w)
        occ, lim, rho = B.moe_query_occupancy(h, tm, tn)
        assert (occ.tile_m, occ.tile_n) == (tm, tn) and occ.comp_slot_sms == (2 if tm == 256 else 1)
        # the co-resident family is offered for the one-CTA tiles (from 24 compute waves on), not for the CTA-pair
        # tiles, where a co-resident warp would cost the seventh operand stage
        assert lim.co_warps_max == 2 and lim.co_min_waves == (2 ** 31 - 1 if tm == 256 else 24)


def test_pair_tiles_against_oracle():
    for kw in (dict(T=777, E=5, k=2, H=1536, I=512, TP=2, EP=3, L=4),      # partial n-tile at the split end
               dict(T=300, E=3, k=1, H=256, I=64, TP=1, EP=1, L=1),         # m-tiles with an empty second half
               dict(T=1030, E=70, k=2, H=512, I=256, TP=2, EP=8, L=2)):     # empty experts
        base = dict(name="pair", routing_seed=3, data_seed=4, tile_m=256, tile_n=256)
        base.update(kw)
        _check_against_oracle(replace(wl.TINY, **base))
    _check_against_oracle(replace(wl.DSV2L, tile_m=256, tile_n=256), n_random=96)


def test_ep_concat_invariance_and_tp_within_tolerance():
    w = replace(wl.QWEN, name="ep", T=1200, E=16)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    cat = {}
    for EP in (1, 2, 4):
        we = replace(w, EP=EP)
        outs, *_ = G.run_layer(we, idx, wt, x, W2)
        cat[EP] = np.concatenate([o[:len(G.tokens_of_rank(w.T, EP, d))] for d, o in enumerate(outs)])
    assert np.array_equal(cat[1], cat[2]) and np.array_equal(cat[1], cat[4])
    expect, _ = _oracle_tokens(w, idx, wt, x, W2)
    for TP in (1, 2, 4):
        wt_ = replace(w, TP=TP)   # K = 1408, 704, 352
        outs, *_ = G.run_layer(wt_, idx, wt, x, W2)
        got = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(outs)])
        assert np.max(np.abs(got - expect)) <= G.tolerance(expect), TP


def test_identity_weights_make_the_combine_exact():
    # W2_e = identity (I = H), small integer activations, power-of-two weights: every partial
    # sum is exactly representable in bf16, so the GPU output must equal the gather exactly
    w = replace(wl.TINY, name="ident", T=300, E=6, k=2, H=128, I=128, TP=1, EP=2, tile_m=64, tile_n=64)
    rng = np.random.default_rng(1)
    idx = np.stack([rng.permutation(w.E)[:2] for _ in range(w.T)]).astype(np.int32)
    wt = np.tile(np.array([0.5, 0.25], dtype=np.float32), (w.T, 1))
    xv = rng.integers(-8, 9, (w.R, w.I)).astype(np.float32)
    x = torch.from_numpy(xv).bfloat16()
    W2 = torch.eye(w.H).repeat(w.E, 1, 1).bfloat16()
    outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2)
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    inv = r["inv_perm"].reshape(w.T, 2)
    expect = 0.5 * xv[inv[:, 0]] + 0.25 * xv[inv[:, 1]]
    got = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(outs)])
    assert np.array_equal(got, expect)


def test_gemm_only_then_combine_only_equals_fused():
    w = replace(wl.GRANITE, name="modes", T=1024)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    fused, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2)
    fused = [o.copy() for o in fused]
    G.run_layer(w, idx, wt, x, W2, mode=B.MOE_MODE_GEMM_ONLY, ws=ws)
    two, *_ = G.run_layer(w, idx, wt, x, W2, mode=B.MOE_MODE_COMBINE_ONLY, ws=ws)
    for a, b in zip(fused, two):
        assert np.array_equal(a, b, equal_nan=True)


def test_a_released_and_rezeroed_flags_workspace_starts_over():
    # the handle keeps the launch epoch of every flags workspace; after moe_release_workspace and a fresh
    # zero-fill the same buffer is a new workspace (epoch 1 again) and gives the same bits
    h = G.handle()
    w = replace(wl.GRANITE, name="release", T=900)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    first, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2)
    first = [o.copy() for o in first]
    G.run_layer(w, idx, wt, x, W2, ws=ws)                     # epoch 2 on the same workspace
    B.moe_release_workspace(h, ws.flags_ws)
    ws.flags_ws.zero_()
    again, *_ = G.run_layer(w, idx, wt, x, W2, ws=ws)
    for a, b in zip(first, again):
        assert np.array_equal(a, b, equal_nan=True)


def test_bounded_wait_reports_a_timeout_and_the_context_survives():
    h = G.handle()
    w = replace(wl.TINY, name="withhold", T=512, E=4, k=2, H=256, I=128, TP=1, EP=1, tile_m=128, tile_n=128)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    mu = r["S"] - 1                                   # the last m-tile: rows of the latest tokens
    n_tiles_n = w.H // w.tile_n
    g_withheld = (mu * w.TP + 0) * n_tiles_n + 0      # (split 0, m-tile mu, shard 0, n-tile 0)
    B.moe_set_wait_limit_ns(h, 20_000_000)            # 20 ms
    try:
        # that tile is computed but its readiness is never raised
        outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2, force_C=2, withhold=g_withheld, check_status=False)
        assert st.code == B.MOE_DEV_TIMEOUT and st.detail == g_withheld and st.where == 40
        # tokens that do not depend on the withheld tile and were served before the wait ran out are correct
        dep = set(int(r["perm"][row]) // w.k_tot
                  for row in range(r["mtile_first_row"][mu], r["mtile_first_row"][mu] + r["mtile_valid"][mu]))
        free = np.array([t for t in range(w.T) if t not in dep], dtype=np.int32)
        expect, _ = _oracle_tokens(w, idx, wt, x, W2, tokens=free)
        got = outs[0][free]
        done = ~np.isnan(got).any(axis=1)            # a CTA that gave up leaves its later rows unwritten
        assert done.sum() >= w.T // 4
        assert np.max(np.abs(got[done] - expect[done])) <= G.tolerance(expect)
    finally:
        B.moe_set_wait_limit_ns(h, 2_000_000_000)
    # the same workspace and context keep working
    outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2, ws=ws)
    assert st.code == 0
    expect, _ = _oracle_tokens(w, idx, wt, x, W2)
    assert np.max(np.abs(outs[0][:w.T] - expect)) <= G.tolerance(expect)


def test_bounded_wait_with_co_resident_warps_winds_down_cleanly():
    # a split that never completes (one readiness flag withheld): the co-resident warps that sleep on its counter
    # and the communication CTAs that poll the tile give up at the limit, the launch returns, the context lives
    h = G.handle()
    w = replace(wl.TINY, name="withhold_co", T=512, E=4, k=2, H=512, I=128, TP=1, EP=1, tile_m=128, tile_n=128, L=2)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    g_withheld = ((r["S"] - 1) * w.TP + 0) * (w.H // w.L // w.tile_n) + 0      # split 0, last m-tile, n-tile 0
    B.moe_set_wait_limit_ns(h, 20_000_000)
    try:
        for tile in ((128, 128), (256, 256)):
            wt_ = replace(w, tile_m=tile[0], tile_n=tile[1])
            gw = g_withheld if tile[0] == 128 else 0
            outs, plan, ws, S, st = G.run_layer(wt_, idx, wt, x, W2, force_C=2, withhold=gw, check_status=False,
                                                drain_help=1, co_warps=2)
            assert plan.co_warps == 2
            assert st.code == B.MOE_DEV_TIMEOUT and st.where in (40, 44)
            outs, plan, ws, S, st = G.run_layer(wt_, idx, wt, x, W2, ws=ws, drain_help=1, co_warps=2)
            assert st.code == 0
            expect, _ = _oracle_tokens(wt_, idx, wt, x, W2)
            assert np.max(np.abs(outs[0][:w.T] - expect)) <= G.tolerance(expect)
    finally:
        B.moe_set_wait_limit_ns(h, 2_000_000_000)


def test_argument_validation():
    h = G.handle()
    w = wl.TINY
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2)
    shape = G.shape_of(w)
    occ, lim, rho = B.moe_query_occupancy(h, w.tile_m, w.tile_n)
    xd, Wd, wd = x.cuda(), W2.cuda(), torch.from_numpy(wt).cuda()
    args = lambda p, xx=xd: (h, xx, Wd, None, wd, shape, occ, ws.routing, S, p, ws.out, ws.y_ws, ws.flags_ws, ws.status)
    # no communication CTA at all is only legal when the compute CTAs serve the communication work themselves
    bad = B.moe_plan.from_buffer_copy(plan); bad.comm_ctas = 0; bad.R = 0; bad.drain_help = 0
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm2_combine(*args(bad))
    assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
    bad = B.moe_plan.from_buffer_copy(plan); bad.comm_ctas = -1
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm2_combine(*args(bad))
    assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
    bad = B.moe_plan.from_buffer_copy(plan); bad.co_warps = 5     # more co-resident warps than a CTA has
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm2_combine(*args(bad))
    assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
    bad = B.moe_plan.from_buffer_copy(plan); bad.P = 148          # C + P > G
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm2_combine(*args(bad))
    assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
    bad = B.moe_plan.from_buffer_copy(plan); bad.R = 0            # reservation too small for C
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm2_combine(*args(bad))
    assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm2_combine(*args(plan, xd.data_ptr() + 2))   # misaligned
    assert e.value.code == B.MOE_ERR_ALIGN
    with pytest.raises(B.MoeError) as e:
        B.moe_gemm2_combine(h, None, Wd, None, wd, shape, occ, ws.routing, S, plan, ws.out, ws.y_ws, ws.flags_ws, ws.status)
    assert e.value.code == B.MOE_ERR_NULL


def test_host_buffer_entry_point_matches_device_path():
    h = G.handle()
    w = replace(wl.GRANITE, name="host", T=1000)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    dev, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2)
    shape = G.shape_of(w)
    nbytes = B.moe_host_arena_bytes(shape, w.tile_m, w.tile_n)
    arena = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    off = (-arena.data_ptr()) % 256
    xh = x.pin_memory(); ih = torch.from_numpy(idx).pin_memory(); wh = torch.from_numpy(wt).pin_memory()
    counts = torch.zeros(w.E_tot + 1, dtype=torch.int32).pin_memory()
    out_h = torch.empty((w.T, w.H), dtype=torch.bfloat16).pin_memory()
    p2 = B.moe_layer_host(h, xh, ih, wh, W2.cuda(), shape, w.tile_m, w.tile_n, None,
                          arena.data_ptr() + off, nbytes, counts, out_h)
    assert (p2.comm_ctas, p2.P) == (plan.comm_ctas, plan.P)
    got = out_h.float().numpy()
    cat = np.concatenate([o[:len(G.tokens_of_rank(w.T, w.EP, d))] for d, o in enumerate(dev)])
    assert np.array_equal(got, cat)


def test_single_call_layer_matches_the_stepwise_path():
    h = G.handle()
    w = replace(wl.GRANITE, name="layer", T=1500)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    ref_outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2)
    ref_outs = [o.copy() for o in ref_outs]
    for o in ws.out:
        o.fill_(float("nan"))
    xd, Wd = x.cuda(), W2.cuda()
    idx_d, wt_d = torch.from_numpy(idx).cuda(), torch.from_numpy(wt).cuda()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(); eb.record()
    call = B.LayerCall(h, xd, Wd, idx_d, wt_d, ws)
    p2 = call(ea, eb)
    torch.cuda.synchronize()
    assert B.moe_get_status(h, ws.status).code == 0
    assert (p2.comm_ctas, p2.P, p2.W_comp) == (plan.comm_ctas, plan.P, plan.W_comp)
    assert ea.elapsed_time(eb) > 0
    for a, o in zip(ref_outs, ws.out):
        assert np.array_equal(a, o.float().cpu().numpy(), equal_nan=True)


@pytest.mark.parametrize("T", [40, 3000, 12000], ids=["one_cta", "cluster", "four_launches"])
def test_whole_step_call_gets_the_counts_of_every_routing_build(T):
    # Section III-E: the manager reads the routed-tile counts on the host between dispatch and launch.  The
    # whole-step call has them written into host memory by the routing kernel and waits for a sequence
    # number; three launch shapes of the routing build (k_tot = 3: 120, 9000 and 36000 assignments), changing
    # routings call after call, counts and outputs against the references every time.
    from oracle import routing_ref as rr
    h = G.handle()
    w = replace(wl.TINY, name="mailed", T=T, E=24, k=3, H=256, I=64, tile_m=128, tile_n=128, EP=2, TP=1, L=2)
    x, W2 = wl.make_data(w)
    xd, Wd = x.cuda(), W2.cuda()
    ws = None
    for rep in range(3):
        wr = replace(w, routing="zipf" if rep else "uniform", zipf_s=1.2, routing_seed=7 + rep)
        idx, wt, _ = wl.make_routing(wr)
        ref_outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2, ws=ws)
        ref_outs = [o.copy() for o in ref_outs]
        ref = rr.build_routing(idx, w.E_tot, w.tile_m)
        for o in ws.out:
            o.fill_(float("nan"))
        ws.tile_counts.fill_(-7)
        idx_d, wt_d = torch.from_numpy(idx).cuda(), torch.from_numpy(wt).cuda()
        p2 = B.moe_layer(h, xd, Wd, idx_d, wt_d, ws)
        # the counts are on the host when the call returns, before any synchronisation by the caller
        assert ws.tile_counts[:w.E_tot].tolist() == ref["tiles"].tolist(), rep
        assert int(ws.tile_counts[w.E_tot]) == ref["S"], rep
        torch.cuda.synchronize()
        assert B.moe_get_status(h, ws.status).code == 0
        assert (p2.comm_ctas, p2.P, p2.W_comp) == (plan.comm_ctas, plan.P, plan.W_comp)
        for a, o in zip(ref_outs, ws.out):
            assert np.array_equal(a, o.float().cpu().numpy(), equal_nan=True), rep


@pytest.mark.parametrize("tile", [(128, 256), (256, 256)], ids=["128x256", "pair"])
def test_counts_left_on_the_device_give_the_same_bits(tile):
    # Section III-E: no copy of the routed counts and no wait; the plan comes from the normalised-load
    # estimate and the kernel reads the m-tile count from the routing workspace.  A skewed routing
    # makes the estimate differ from the true tile count; the output may not change by a bit.
    h = G.handle()
    w = replace(wl.DSV2L, name="devcounts", T=3000, tile_m=tile[0], tile_n=tile[1])
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    ref_outs, plan, ws, S, st = G.run_layer(w, idx, wt, x, W2)
    ref_outs = [o.copy() for o in ref_outs]
    xd, Wd = x.cuda(), W2.cuda()
    idx_d, wt_d = torch.from_numpy(idx).cuda(), torch.from_numpy(wt).cuda()
    for rep in range(2):
        for o in ws.out:
            o.fill_(float("nan"))
        ws.tile_counts.fill_(-7)                       # must stay untouched
        p2 = B.moe_layer(h, xd, Wd, idx_d, wt_d, ws, counts_on_device=True)
        torch.cuda.synchronize()
        assert B.moe_get_status(h, ws.status).code == 0
        assert (ws.tile_counts == -7).all()
        occ, lim, rho = B.moe_query_occupancy(h, w.tile_m, w.tile_n)
        est = B.plan_partition_estimate(occ, lim, ws.shape, rho)
        assert (p2.comm_ctas, p2.P, p2.W_comp) == (est.comm_ctas, est.P, est.W_comp)
        assert p2.W_comp != plan.W_comp                # the estimate is not the true count here
        for a, o in zip(ref_outs, ws.out):
            assert np.array_equal(a, o.float().cpu().numpy(), equal_nan=True), rep


def test_service_rate_characterisation_entry_point():
    # Eq. 13 through the library: a positive, finite rho_ref with the reference factors of the workload
    # it ran on, the device status clean, and two calls that agree within the run-to-run spread
    h = G.handle()
    w = replace(wl.DSV2L, name="rho_ref", T=2048, routing="uniform", zipf_s=0.0, target_r_expert=0.0,
                tile_m=128, tile_n=256)
    idx, wt, _ = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    ws, idx_d, S = G.build_routing(w, idx, None)
    xd, Wd, wt_d = x.cuda(), W2.cuda(), torch.from_numpy(wt).cuda()
    vals = []
    for _ in range(2):
        rho, wave_comp, wave_comm = B.moe_calibrate_rho(h, xd, Wd, idx_d, wt_d, ws, C_ref=32, n_samples=7)
        assert B.moe_get_status(h, ws.status).code == 0
        assert wave_comp > 0 and wave_comm > 0 and abs(rho.rho_ref - wave_comm / wave_comp) < 1e-9
        assert (rho.K_ref, rho.tile_m_ref, rho.tile_n_ref, rho.D_ref) == (w.K, 128, 256, w.EP)
        assert rho.rows_ref == w.k_tot * w.TP + 1 and rho.comm_cols_ref == 1024
        assert 1.0 < rho.rho_ref < 200.0
        vals.append(rho.rho_ref)
    assert abs(vals[0] - vals[1]) / vals[0] < 0.3
    with pytest.raises(B.MoeError):
        B.moe_calibrate_rho(h, xd, Wd, idx_d, wt_d, ws, C_ref=0)


def test_random_small_shapes_against_the_oracle():
    # seeded fuzz over the argument space the kernels accept: tile families, splits, shards, ranks, ragged
    # sizes, forced and analytical C, static map and dynamic hand-out; every token checked
    rng = np.random.default_rng(2024)
    n_done = 0
    for case in range(36):
        tile_m, tile_n = [(64, 64), (64, 128), (128, 64), (128, 128), (128, 256), (256, 256)][int(rng.integers(6))]
        TP = int(rng.choice([1, 2, 4]))
        K = int(rng.choice([16, 48, 64, 80, 128, 208]))
        L = int(rng.choice([1, 2, 3, 4]))
        H = int(rng.choice([64, 136, 256, 320, 768])) * L if rng.random() < 0.5 else int(rng.choice([64, 128, 264, 512, 1024]))
        if (-(-H // L)) % 8 != 0 or H % 8 != 0:
            continue
        E = int(rng.integers(1, 20))
        k = int(rng.integers(1, min(E, 4) + 1))
        n_shared = int(rng.choice([0, 0, 1, 2]))
        T = int(rng.choice([1, 7, 65, 200, 513, 900]))
        EP = int(rng.choice([1, 2, 3, 4, 8]))
        w = replace(wl.TINY, name=f"fuzz{case}", T=T, H=H, I=K * TP, E=E, k=k, n_shared=n_shared, TP=TP, EP=EP, L=L,
                    tile_m=tile_m, tile_n=tile_n, routing="zipf" if rng.random() < 0.5 else "uniform",
                    zipf_s=1.0, target_r_expert=0.0, routing_seed=100 + case, data_seed=200 + case)
        kw = dict(drain_help=int(rng.integers(2)))
        if rng.random() < 0.5:
            kw["force_C"] = int(rng.choice([1, 2, 5, 33]))
        _check_against_oracle(w, **kw)
        n_done += 1
    assert n_done >= 25


def test_random_small_shapes_with_co_resident_warps_against_the_oracle():
    # the same fuzz with co-resident communication warps asked for (the launch drops them where the shape has no
    # room for them), with and without dedicated communication CTAs; every token checked
    rng = np.random.default_rng(2025)
    n_done = 0
    for case in range(30):
        tile_m, tile_n = [(64, 64), (128, 64), (128, 128), (128, 256), (256, 256)][int(rng.integers(5))]
        TP = int(rng.choice([1, 2, 4]))
        K = int(rng.choice([16, 64, 80, 128, 208]))
        L = int(rng.choice([1, 2, 2, 4]))
        H = int(rng.choice([64, 128, 256, 320, 512])) * L
        E = int(rng.integers(1, 20))
        k = int(rng.integers(1, min(E, 4) + 1))
        n_shared = int(rng.choice([0, 0, 1, 2]))
        T = int(rng.choice([1, 7, 65, 200, 513, 900, 1500]))
        EP = int(rng.choice([1, 2, 3, 4]))
        w = replace(wl.TINY, name=f"cofuzz{case}", T=T, H=H, I=K * TP, E=E, k=k, n_shared=n_shared, TP=TP, EP=EP, L=L,
                    tile_m=tile_m, tile_n=tile_n, routing="zipf" if rng.random() < 0.5 else "uniform",
                    zipf_s=1.0, target_r_expert=0.0, routing_seed=300 + case, data_seed=400 + case)
        kw = dict(drain_help=1, co_warps=int(rng.choice([1, 2])))
        r = rng.random()
        if r < 0.35:
            kw["force_C"] = int(rng.choice([1, 2, 5, 33]))
        elif r < 0.6:      # no dedicated communication CTA at all: every SM computes
            kw.update(force_C=1, C_override=0, P_override=148 // (2 if tile_m == 256 else 1))
        _check_against_oracle(w, **kw)
        n_done += 1
    assert n_done >= 25
