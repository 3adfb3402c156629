"""plan_partition (library, host C++) against the selector reference: bit-exact on every
field, over random inputs, the BASELINE shapes, the overrides and the error paths."""

import random
import time

import numpy as np
import pytest

from oracle import routing_ref as rr
from oracle import solver_ref as sr
from paper_2609_07536_b200 import binding as B
from paper_2609_07536_b200 import workloads as wl


def _oracle_plan(tiles, shape, occ, lim, rho):
    K = shape.I // shape.TP
    Wc = sr.w_comp(tiles, shape.TP, shape.H, shape.L, occ.tile_n)
    Wm = sr.w_comm_gpu(shape.T, shape.EP, shape.H, shape.L, occ.comm_tile_m, occ.comm_tile_n)
    if rho.mode == B.MOE_RHO_PAPER:
        r = sr.rho_scaled(rho.rho_ref, rho.K_ref, rho.tile_m_ref, rho.tile_n_ref, rho.D_ref,
                          K, occ.tile_m, occ.tile_n, shape.EP)
    else:
        r = sr.rho_local(rho.rho_ref, rho.K_ref, rho.tile_m_ref, rho.tile_n_ref, rho.rows_ref,
                         rho.comm_cols_ref, K, occ.tile_m, occ.tile_n, shape.k_tot, shape.TP,
                         shape.H, shape.L, occ.comm_tile_n)
    rho_q = sr.quantise_rho(r)
    if lim.drain_help and rho.comm_warps_per_cta > 0:
        # the co-resident family: product set (C, w), bandwidth-coupled service rate
        sel = sr.select_co_resident(
            Wc, Wm, shape.L, lim.G, occ.o_comp, occ.o_comm, lim.C_max, rho_q, occ.comp_slot_sms,
            max(0, lim.co_warps_max), lim.C_co_max, rho.comm_warps_per_cta,
            rho.n_sat_warps if rho.n_sat_warps > 0 else 2 ** 63 - 1, sr.quantise_rho(rho.co_beta),
            sr.quantise_rho(rho.co_gamma), sr.quantise_rho(rho.co_order), force_comm_ctas=lim.force_comm_ctas,
            selector_off=bool(lim.selector_off), default_C=lim.default_C, force_co_warps=lim.force_co_warps,
            quanta_tile=rho.comm_quanta_per_tile, co_min_waves=lim.co_min_waves)
    elif not lim.drain_help and lim.dep_model == B.MOE_DEP_TILE:
        # static partition with tile-level readiness
        idx = sr.comm_tile_ready_index(tiles, shape.TP, shape.T, shape.EP, shape.H, shape.L, occ.tile_n,
                                       occ.comm_tile_m, occ.comm_tile_n)
        assert len(idx) == Wm
        if lim.force_comm_ctas > 0 or lim.selector_off:
            Cs = [lim.force_comm_ctas if lim.force_comm_ctas > 0 else lim.default_C]
            if Cs[0] < 1:
                raise ValueError("C must be at least 1")
        else:
            Cs = range(1, lim.C_max + 1)
        best = None
        for C in Cs:
            m = sr.makespan_tile_level(C, idx, Wc, shape.L, lim.G, occ.o_comp, occ.o_comm, rho_q, occ.comp_slot_sms)
            if m is not None and (best is None or (m[0], m[1], C) < best[0]):
                best = ((m[0], m[1], C), dict(comm_ctas=C, R=m[2], P=m[3], T_q=m[0], delta=m[1], W_comp=Wc, W_comm=Wm))
        if best is None:
            raise ValueError("no legal C")
        sel = best[1]
    else:
        sel = sr.select(Wc, Wm, shape.L, lim.G, occ.o_comp, occ.o_comm, lim.C_max, rho_q,
                        force_comm_ctas=lim.force_comm_ctas, selector_off=bool(lim.selector_off),
                        default_C=lim.default_C, slot_sms=occ.comp_slot_sms, drain_help=bool(lim.drain_help))
        if lim.drain_help and lim.co_warps_max > 0 and lim.force_co_warps > 0:
            sel["co_warps"] = min(lim.force_co_warps, lim.co_warps_max)   # an explicit request is passed through
    sel.setdefault("co_warps", 0)
    sel["rho_q"] = rho_q
    return sel


def _same(plan, sel):
    assert (plan.comm_ctas, plan.R, plan.P) == (sel["comm_ctas"], sel["R"], sel["P"])
    assert (plan.W_comp, plan.W_comm, plan.delta) == (sel["W_comp"], sel["W_comm"], sel["delta"])
    assert plan.pred_T_q == sel["T_q"] and plan.rho_q == sel["rho_q"]
    assert plan.mode == B.MOE_MODE_FUSED and plan.debug_withhold_tile == -1 and plan.co_warps == sel["co_warps"]


def _rand_inputs(rng):
    E = rng.choice([1, 8, 40, 66])
    tile_m = rng.choice([64, 128])
    tile_n = rng.choice([64, 128, 256])
    TP = rng.choice([1, 2, 4])
    shape = B.make_shape(rng.choice([1, 37, 256, 4096, 16384, 32768]), rng.choice([256, 1536, 2048, 4096]),
                         rng.choice([128, 512, 1408]) * TP, E, rng.choice([1, 2, 8]), TP,
                         rng.choice([1, 2, 4, 8]), rng.choice([1, 2, 4, 8]))
    occ = B.moe_occupancy(tile_m, tile_n, rng.choice([64, 128]), rng.choice([512, 1024]),
                          rng.choice([1, 2]), rng.choice([1, 2, 4]), rng.choice([1, 1, 2]))
    # the three model families: the paper's recurrence / drain help (as before), the co-resident family with
    # a bandwidth-coupled service rate (drain help and warp-level constants), tile-level readiness (static)
    family = rng.choice(["plain", "plain", "co", "co", "tile"])
    dh = 1 if family == "co" else (0 if family == "tile" else rng.choice([0, 0, 1]))
    lim = B.moe_sm_limits(rng.choice([4, 108, 148]), rng.randint(1, 160), 0, 0, 3, dh,
                          rng.choice([0, 1, 2, 4]), rng.choice([-1, -1, 0, 1, 3]), rng.choice([1, 8, 16, 200]),
                          B.MOE_DEP_TILE if family == "tile" else rng.choice([B.MOE_DEP_SPLIT, B.MOE_DEP_TILE]),
                          rng.choice([0, 0, 5, 24, 300]))
    rho = B.moe_rho(rng.uniform(0.05, 30.0), rng.choice([352, 704]), 128, rng.choice([128, 256]),
                    rng.choice([2, 4]), 17, 1024, rng.choice([B.MOE_RHO_PAPER, B.MOE_RHO_LOCAL]))
    if family == "co":
        rho.comm_warps_per_cta = rng.choice([1, 4, 12])
        rho.n_sat_warps = rng.choice([0, 7, 300, 1030, 100000])
        rho.comm_quanta_per_tile = rng.choice([0, 0, 12, 128, 5])
        rho.co_beta = rng.choice([0.0, 0.0125, 0.2])
        rho.co_gamma = rng.choice([1.0, 2.2, 7.5])
        rho.co_order = rng.choice([0.0, 0.02, 0.3])
    tiles = [rng.randint(0, 40) for _ in range(E)]
    return tiles, shape, occ, lim, rho


def test_random_inputs_bit_exact():
    rng = random.Random(11)
    n = 0
    for _ in range(100000):
        tiles, shape, occ, lim, rho = _rand_inputs(rng)
        try:
            sel = _oracle_plan(tiles, shape, occ, lim, rho)
        except ValueError:
            with pytest.raises(B.MoeError) as e:
                B.plan_partition(tiles, occ, lim, shape, rho)
            assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
            continue
        _same(B.plan_partition(tiles, occ, lim, shape, rho), sel)
        n += 1
    assert n > 75000


def test_overrides_and_errors():
    rng = random.Random(12)
    for _ in range(2000):
        tiles, shape, occ, lim, rho = _rand_inputs(rng)
        lim.force_comm_ctas = rng.choice([0, 0, 1, 5, 200])
        lim.selector_off = rng.choice([0, 1])
        lim.default_C = rng.choice([1, 3, 16, 500])
        try:
            sel = _oracle_plan(tiles, shape, occ, lim, rho)
        except ValueError:
            with pytest.raises(B.MoeError) as e:
                B.plan_partition(tiles, occ, lim, shape, rho)
            assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
            continue
        plan = B.plan_partition(tiles, occ, lim, shape, rho)
        _same(plan, sel)
        if lim.force_comm_ctas > 0:
            assert plan.comm_ctas == lim.force_comm_ctas      # the user's C wins over everything
        elif lim.selector_off:
            assert plan.comm_ctas == lim.default_C
    # argument errors
    tiles, shape, occ, lim, rho = _rand_inputs(random.Random(1))
    assert B.lib().plan_partition(None, 0, None, None, None, None, None) == B.MOE_ERR_NULL
    bad = B.make_shape(16, 256, 128, 8, 2, 1, 2, 0)
    with pytest.raises(B.MoeError) as e:
        B.plan_partition(tiles, occ, lim, bad, rho)
    assert e.value.code == B.MOE_ERR_SHAPE
    with pytest.raises(B.MoeError):
        B.plan_partition([-1] * shape.E_tot, occ, lim, shape, rho)


@pytest.mark.parametrize("w", [wl.TINY, wl.GRANITE, wl.QWEN, wl.DSV2L], ids=lambda w: w.name)
def test_baseline_shapes(w):
    idx, _, _ = wl.make_routing(w)
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    shape = B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
    occ = B.moe_occupancy(w.tile_m, w.tile_n, 128, 1024, 1, 1, 1)
    lim = B.moe_sm_limits(148, 74, 0, 0, 3)
    for mode in (B.MOE_RHO_PAPER, B.MOE_RHO_LOCAL):
        rho = B.moe_rho(2.5, 704, 128, 256, 2, 17, 1024, mode)
        plan = B.plan_partition(r["tiles"].tolist(), occ, lim, shape, rho)
        _same(plan, _oracle_plan(r["tiles"].tolist(), shape, occ, lim, rho))
        assert 1 <= plan.comm_ctas <= 74 and plan.P == 148 - plan.R and plan.R == plan.comm_ctas
        assert plan.W_comp == w.TP * r["S"] * -(-(-(-w.H // w.L)) // w.tile_n)


def test_golden_examples_through_the_library(golden_dir):
    # Ex.C and Ex.D of the hand-worked examples, expressed as library inputs
    # Ex.C: W_comp = 8192 = TP 2 x S 1024 x 4 n-tiles ; W_comm = 64 (one rank of 8192 tokens)
    shape = B.make_shape(8192, 2048, 1408, 64, 8, 2, 1, 2)
    occ = B.moe_occupancy(128, 256, 128, 1024, 1, 1, 1)
    lim = B.moe_sm_limits(148, 74, 0, 0, 3)
    rho = B.moe_rho(3.0, 704, 128, 256, 1, 17, 1024, B.MOE_RHO_PAPER)
    plan = B.plan_partition([16] * 64, occ, lim, shape, rho)
    assert (plan.W_comp, plan.W_comm) == (8192, 64)
    assert (plan.comm_ctas, plan.R, plan.P, plan.delta) == (13, 13, 135, 43)
    assert plan.pred_T_q == 137 << 20 and plan.rho_q == 3145728
    # Ex.D: o_comm = 2, W_comp = 1000 = 1 x 1000 x 1, W_comm = 37, L = 4, rho = 2.5
    shape = B.make_shape(37 * 128, 1024, 704, 10, 8, 1, 1, 4)
    occ = B.moe_occupancy(128, 256, 128, 1024, 1, 2, 1)
    lim = B.moe_sm_limits(148, 32, 0, 0, 3)
    rho = B.moe_rho(2.5, 704, 128, 256, 1, 17, 1024, B.MOE_RHO_PAPER)
    plan = B.plan_partition([100] * 10, occ, lim, shape, rho)
    assert (plan.W_comp, plan.W_comm) == (1000, 37)
    assert (plan.comm_ctas, plan.R, plan.P, plan.delta) == (19, 10, 138, 104)
    assert plan.pred_T_q == 34 << 20


def test_pair_slots():
    # a compute slot that spans two SMs (CTA pair): P(C) = floor((G - C) / 2); an odd C strands one SM
    shape = B.make_shape(16384, 2048, 1408, 66, 8, 2, 2, 2)
    occ = B.moe_occupancy(256, 256, 128, 1024, 1, 1, 2)
    rho = B.moe_rho(9.0, 704, 128, 256, 2, 17, 1024, B.MOE_RHO_LOCAL)
    for C in (1, 2, 7, 20, 146, 147):
        lim = B.moe_sm_limits(148, 74, C, 0, 3)
        if (148 - C) // 2 < 1:
            with pytest.raises(B.MoeError):
                B.plan_partition([8] * 66, occ, lim, shape, rho)
            continue
        plan = B.plan_partition([8] * 66, occ, lim, shape, rho)
        assert plan.P == (148 - C) // 2 and plan.R == C
        _same(plan, _oracle_plan([8] * 66, shape, occ, lim, rho))
    lim = B.moe_sm_limits(148, 74, 0, 0, 3)
    plan = B.plan_partition([8] * 66, occ, lim, shape, rho)
    assert plan.comm_ctas % 2 == 0           # an odd C never beats the even one below it by the model


def test_a_family_closed_by_its_lower_bound_is_never_picked_but_a_forced_w_is_honoured():
    # Section III-E (legal set from a one-time characterisation): for the CTA-pair tiles the library hands out
    # co_min_waves = INT32_MAX, i.e. the co-resident family is not offered; a forced w bypasses the bound.
    shape = B.make_shape(16384, 2048, 1408, 66, 8, 2, 2, 2)
    occ = B.moe_occupancy(256, 256, 128, 1024, 1, 1, 2)
    rho = B.moe_rho(14.96, 704, 256, 256, 2, 17, 1024, B.MOE_RHO_LOCAL)
    rho.comm_warps_per_cta, rho.n_sat_warps, rho.comm_quanta_per_tile = 12, 1030, 128
    rho.co_beta, rho.co_gamma, rho.co_order = 0.0125, 2.2, 0.02
    tiles = [8] * 64 + [32] * 2
    picks = {}
    for waves in (24, 2 ** 31 - 1):
        lim = B.moe_sm_limits(148, 74, 0, 0, 3, 1, 2, -1, 8, B.MOE_DEP_SPLIT, waves)
        plan = B.plan_partition(tiles, occ, lim, shape, rho)
        _same(plan, _oracle_plan(tiles, shape, occ, lim, rho))
        picks[waves] = plan
    assert picks[24].co_warps > 0                      # offered, the model takes it on this workload
    assert picks[2 ** 31 - 1].co_warps == 0            # closed: only (C, 0) candidates are left
    lim = B.moe_sm_limits(148, 74, 0, 0, 3, 1, 2, 2, 8, B.MOE_DEP_SPLIT, 2 ** 31 - 1)
    plan = B.plan_partition(tiles, occ, lim, shape, rho)
    _same(plan, _oracle_plan(tiles, shape, occ, lim, rho))
    assert plan.co_warps == 2


def test_drain_help_model():
    # the extension: after the last compute wave every SM serves communication tiles
    shape = B.make_shape(16384, 2048, 1408, 66, 8, 2, 2, 4)
    occ = B.moe_occupancy(128, 256, 128, 1024, 1, 1, 1)
    rho = B.moe_rho(9.0, 704, 128, 256, 2, 17, 1024, B.MOE_RHO_LOCAL)
    tiles = [17] * 66
    picks = {}
    for dh in (0, 1):
        lim = B.moe_sm_limits(148, 74, 0, 0, 3, dh)
        plan = B.plan_partition(tiles, occ, lim, shape, rho)
        _same(plan, _oracle_plan(tiles, shape, occ, lim, rho))
        assert plan.drain_help == dh
        picks[dh] = plan
    # on this workload the helpers shorten the predicted tail and the selector asks for fewer communication CTAs
    assert picks[1].pred_T_q <= picks[0].pred_T_q and picks[1].comm_ctas <= picks[0].comm_ctas
    # closed form for L = 1: T = A_0 + rho * ceil(W_comm / (C + P))
    shape1 = B.make_shape(4096, 2048, 1408, 66, 8, 2, 1, 1)
    lim = B.moe_sm_limits(148, 74, 10, 0, 3, 1)
    plan = B.plan_partition(tiles, occ, lim, shape1, rho)
    A0 = -(-plan.W_comp // plan.P)
    assert plan.pred_T_q == (A0 << 20) + plan.rho_q * -(-plan.W_comm // (10 + plan.P))


def test_solver_cost_is_small():
    # not a benchmark: only guards against an accidental blow-up (ctypes overhead dominates here)
    w = wl.DSV2L
    shape = B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
    occ = B.moe_occupancy(128, 256, 128, 1024, 1, 1, 1)
    lim = B.moe_sm_limits(148, 74, 0, 0, 3)
    rho = B.moe_rho(2.5, 704, 128, 256, 2, 17, 1024, B.MOE_RHO_LOCAL)
    tiles = [17] * 66
    t = time.perf_counter()
    for _ in range(2000):
        B.plan_partition(tiles, occ, lim, shape, rho)
    assert (time.perf_counter() - t) / 2000 < 1e-3


def test_estimate_plan_equals_the_oracle_on_the_normalised_counts():
    # Section III-E, counts left on the device: the library's estimate is the oracle's, and the plan on
    # it is bit-exact like any other
    rng = random.Random(21)
    n = 0
    for _ in range(3000):
        _, shape, occ, lim, rho = _rand_inputs(rng)
        tiles = sr.normalised_load_tiles(shape.T, shape.k_tot, shape.E_tot, occ.tile_m)
        try:
            sel = _oracle_plan(tiles, shape, occ, lim, rho)
        except ValueError:
            with pytest.raises(B.MoeError) as e:
                B.plan_partition_estimate(occ, lim, shape, rho)
            assert e.value.code == B.MOE_ERR_PLAN_INFEASIBLE
            continue
        _same(B.plan_partition_estimate(occ, lim, shape, rho), sel)
        n += 1
    assert n > 2000
