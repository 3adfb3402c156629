"""Pins for the routing reference: invariants, brute force on tiny inputs, degenerate cases.

None of these re-types the reference's own loops: each checks a property that the
definition (a stable sort of the flat assignments by expert, ceil(M_e/T_M) tiles per expert)
fixes independently.
"""

import numpy as np
import pytest

from oracle import routing_ref as rr
from paper_2609_07536_b200 import workloads as wl


def _check_invariants(idx, E_tot, tile_m, r):
    T, k_tot = idx.shape
    R = T * k_tot
    flat = idx.reshape(-1)
    # permutation o inverse = identity, both ways
    assert np.array_equal(r["perm"][r["inv_perm"]], np.arange(R))
    assert np.array_equal(r["inv_perm"][r["perm"]], np.arange(R))
    # counts agree with an independent histogram and sum to R
    assert np.array_equal(r["counts"], np.bincount(flat, minlength=E_tot))
    assert int(r["counts"].sum()) == R and int(r["offsets"][-1]) == R
    # rows of one expert are contiguous, and ascending in f inside it (stability)
    experts_of_rows = flat[r["perm"]]
    assert np.all(np.diff(experts_of_rows) >= 0)
    same = np.diff(experts_of_rows) == 0
    assert np.all(np.diff(r["perm"])[same] > 0)
    # numpy's stable argsort is the same permutation
    assert np.array_equal(r["perm"], np.argsort(flat, kind="stable"))
    # tile bounds:  ceil(R/T_M) <= S <= floor(R/T_M) + #non-empty experts
    S = r["S"]
    nonempty = int((r["counts"] > 0).sum())
    assert -(-R // tile_m) <= S <= R // tile_m + nonempty
    assert S == int(r["tiles"].sum()) == int(r["tile_offsets"][-1])
    # m-tile table: the valid rows of an expert's tiles add up to M_e and tile the segment
    for e in range(E_tot):
        mus = np.arange(r["tile_offsets"][e], r["tile_offsets"][e + 1])
        assert np.all(r["mtile_expert"][mus] == e)
        assert int(r["mtile_valid"][mus].sum()) == int(r["counts"][e])
        if len(mus):
            assert np.array_equal(r["mtile_first_row"][mus], r["offsets"][e] + tile_m * np.arange(len(mus)))
            assert np.all(r["mtile_valid"][mus][:-1] == tile_m)
            assert 1 <= r["mtile_valid"][mus][-1] <= tile_m
    # padded rows: injective, inside the tile that the m-tile table names
    pr = r["pad_row"]
    assert len(np.unique(pr)) == R
    mu = pr // tile_m
    assert np.all(r["mtile_expert"][mu] == flat)
    assert np.array_equal(r["mtile_first_row"][mu] + pr % tile_m, r["inv_perm"])
    assert np.all(pr % tile_m < r["mtile_valid"][mu])


@pytest.mark.parametrize("w", [wl.TINY, wl.GRANITE, wl.DSV2L], ids=lambda w: w.name)
def test_invariants_on_configs(w):
    idx, wt, _ = wl.make_routing(w)
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    _check_invariants(idx, w.E_tot, w.tile_m, r)
    assert r["S"] >= -(-w.R // w.tile_m)


def test_brute_force_tiny():
    rng = np.random.default_rng(5)
    T, k, E = 23, 3, 7
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    r = rr.build_routing(idx, E, 4)
    for f in range(T * k):
        assert r["inv_perm"][f] == rr.brute_force_row(idx, f)
    _check_invariants(idx, E, 4, r)


def test_hand_example():
    # 3 tokens, top-2, 3 experts, tile 2: worked by hand.
    idx = np.array([[2, 0], [0, 1], [2, 1]], dtype=np.int32)
    # flat f: 0:e2 1:e0 2:e0 3:e1 4:e2 5:e1 ; sorted rows: e0:[1,2] e1:[3,5] e2:[0,4]
    r = rr.build_routing(idx, 3, 2)
    assert r["counts"].tolist() == [2, 2, 2]
    assert r["offsets"].tolist() == [0, 2, 4, 6]
    assert r["perm"].tolist() == [1, 2, 3, 5, 0, 4]
    assert r["inv_perm"].tolist() == [4, 0, 1, 2, 5, 3]
    assert r["tiles"].tolist() == [1, 1, 1] and r["S"] == 3
    assert r["pad_row"].tolist() == [4, 0, 1, 2, 5, 3]
    # tile 4: each expert gets one padded tile of 4 rows
    r4 = rr.build_routing(idx, 3, 4)
    assert r4["pad_row"].tolist() == [8, 0, 1, 4, 9, 5]
    assert r4["mtile_valid"].tolist() == [2, 2, 2]
    assert r4["mtile_first_row"].tolist() == [0, 2, 4]


def test_degenerate_cases():
    # all tokens to one expert; other experts empty
    idx = np.full((10, 1), 3, dtype=np.int32)
    r = rr.build_routing(idx, 5, 4)
    assert r["counts"].tolist() == [0, 0, 0, 10, 0]
    assert r["tiles"].tolist() == [0, 0, 0, 3, 0] and r["S"] == 3
    assert r["perm"].tolist() == list(range(10))
    assert r["mtile_valid"].tolist() == [4, 4, 2]
    _check_invariants(idx, 5, 4, r)
    # E = 1, k = 1
    r = rr.build_routing(np.zeros((7, 1), dtype=np.int32), 1, 8)
    assert r["S"] == 1 and r["mtile_valid"].tolist() == [7]
    # exact multiple of the tile: no partial tile
    r = rr.build_routing(np.zeros((8, 1), dtype=np.int32), 1, 4)
    assert r["mtile_valid"].tolist() == [4, 4]
    # empty input
    r = rr.build_routing(np.zeros((0, 2), dtype=np.int32), 4, 4)
    assert r["S"] == 0 and r["counts"].tolist() == [0, 0, 0, 0]


def test_rejects_bad_input():
    with pytest.raises(ValueError):
        rr.build_routing(np.array([[0, 5]], dtype=np.int32), 4, 4)
    with pytest.raises(ValueError):
        rr.build_routing(np.array([[0, -1]], dtype=np.int32), 4, 4)
    with pytest.raises(ValueError):
        rr.build_routing(np.array([[1, 1]], dtype=np.int32), 4, 4)


def test_workload_conventions():
    # generator conventions the routing order relies on: weights sum to 1 over the routed
    # slots, shared experts carry weight exactly 1 and ids E, E+1
    for w in (wl.TINY, wl.DSV2L):
        idx, wt, info = wl.make_routing(w)
        assert idx.shape == (w.T, w.k_tot) and wt.dtype == np.float32
        assert np.allclose(wt[:, :w.k].sum(axis=1), 1.0, atol=1e-6)
        assert np.all(np.diff(wt[:, :w.k], axis=1) <= 0)       # descending logits
        if w.n_shared:
            assert np.all(wt[:, w.k:] == 1.0)
            assert np.all(idx[:, w.k:] == np.arange(w.E, w.E_tot))
    _, _, info = wl.make_routing(wl.DSV2L)
    assert abs(info["r_expert"] - 3.0) < 0.15
    _, _, info = wl.make_routing(wl.GRANITE)
    assert abs(info["r_expert"] - 2.5) < 0.125
