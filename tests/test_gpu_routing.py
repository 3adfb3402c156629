"""GPU routing builder against the routing reference: every array bit-exact."""

import numpy as np
import pytest
import torch

from oracle import routing_ref as rr
from paper_2609_07536_b200 import binding as B
from paper_2609_07536_b200 import workloads as wl
from tests import gpu_common as G

pytestmark = pytest.mark.gpu

KEYS = ["counts", "offsets", "tiles", "tile_offsets", "perm", "inv_perm", "pad_row",
        "mtile_expert", "mtile_first_row", "mtile_valid"]


def _compare(w, idx):
    ws, _, S = G.build_routing(w, idx)
    st = B.moe_get_status(G.handle(), ws.status)
    assert st.code == 0
    ref = rr.build_routing(idx, w.E_tot, w.tile_m)
    assert S == ref["S"]
    got = G.routing_to_numpy(ws, S)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), k
    assert ws.tile_counts[:w.E_tot].tolist() == ref["tiles"].tolist()


@pytest.mark.parametrize("w", [wl.TINY, wl.GRANITE, wl.QWEN, wl.DSV2L], ids=lambda w: w.name)
def test_configs(w):
    idx, _, _ = wl.make_routing(w)
    _compare(w, idx)


def test_adversarial():
    from dataclasses import replace
    base = replace(wl.TINY, T=300, E=9, k=1, tile_m=64)
    # one hot expert, others empty
    _compare(base, np.full((300, 1), 4, dtype=np.int32))
    # E = 1
    _compare(replace(base, E=1), np.zeros((300, 1), dtype=np.int32))
    # T not a tile multiple, k = 3, tile 128, many empty experts
    rng = np.random.default_rng(0)
    w = replace(wl.TINY, T=1001, E=70, k=3, tile_m=128)
    idx = np.stack([rng.choice(13, 3, replace=False) * 5 for _ in range(1001)]).astype(np.int32)
    _compare(w, idx)
    # a single token
    _compare(replace(base, T=1, E=4, k=2), np.array([[3, 0]], dtype=np.int32))
    # the sweep's largest size
    big = wl.sweep_workloads(T_list=(32768,), s_list=(1.2,), EP_list=(4,), tiles=((128, 256),))[0]
    idx, _, _ = wl.make_routing(big)
    _compare(big, idx)


def test_batches_of_the_cluster_launch():
    """33 to 128 chunks of 256 assignments go through one cluster of 8 CTAs: uneven chunk runs (a CTA with
    fewer chunks, a CTA with none), a ragged last chunk, one hot expert, bad ids reported."""
    from dataclasses import replace
    rng = np.random.default_rng(3)
    for T, E, k, tm in ((2817, 40, 3, 128),      # 8451 assignments: 34 chunks, CTA 7 of 8 gets none
                        (9003, 66, 1, 64),       # 36 chunks, the last one ragged
                        (4099, 256, 8, 256),     # 129 chunks: the first size of the four-launch path
                        (4000, 200, 8, 128)):    # 125 chunks, many experts
        w = replace(wl.TINY, T=T, E=E, k=k, tile_m=tm, tile_n=256 if tm == 256 else 64)
        idx = np.stack([rng.choice(E, k, replace=False) for _ in range(T)]).astype(np.int32)
        _compare(w, idx)
    w = replace(wl.TINY, T=10000, E=9, k=1, tile_m=64)
    _compare(w, np.full((10000, 1), 4, dtype=np.int32))
    idx = rng.integers(0, 9, size=(10000, 1)).astype(np.int32)
    bad = idx.copy()
    bad[9000, 0] = -3
    ws, _, S = G.build_routing(w, bad)
    st = B.moe_get_status(G.handle(), ws.status, check=False)
    assert st.code == B.MOE_DEV_OOB and st.detail == 9000
    _compare(w, idx)


def test_bad_ids_are_reported_not_fatal():
    from dataclasses import replace
    w = replace(wl.TINY, T=64, E=8, k=2)
    idx, _, _ = wl.make_routing(w)
    bad = idx.copy()
    bad[5, 1] = 99
    ws, _, S = G.build_routing(w, bad)
    st = B.moe_get_status(G.handle(), ws.status, check=False)
    assert st.code == B.MOE_DEV_OOB and st.detail == 5 * 2 + 1
    dup = idx.copy()
    dup[7, 1] = dup[7, 0]
    ws, _, S = G.build_routing(w, dup)
    st = B.moe_get_status(G.handle(), ws.status, check=False)
    assert st.code == B.MOE_DEV_DUP_EXPERT and st.detail == 7
    # the context is still usable
    _compare(w, idx)
