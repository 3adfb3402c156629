"""Routing / permutation / routed-tile-count reference (CPU oracle, test infrastructure).

This file is test infrastructure: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it.  It shares no code with the CUDA path.

What it computes (paper Section II-A "Distributed MoE Execution": the router yields
token-expert assignments; Section III-C Eq. 5: expert e needs ceil(M_e / T_M) tiles along
the token dimension; Section III-E Eq. 16: the host reduces the routed counts to
sum_e ceil(M_e / T_M)).  The paper fixes no ordering of the routed rows, so the reading
taken here is the usual one: a *stable* sort of the flat assignment ids by expert.

Everything is written as plain loops over python ints so that it can be read against the
definitions; it is O(R) and finishes in well under a second at R = 131072.
"""

from __future__ import annotations

import numpy as np


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def build_routing(topk_idx, E_tot: int, tile_m: int) -> dict:
    """Plain-loop routing reference.

    topk_idx : int array [T, k_tot]; entry [t, j] is the expert of flat assignment
               f = t * k_tot + j.
    Returns a dict of int32 numpy arrays:
      counts[e]        M_e, assignments received by expert e
      offsets[e]       exclusive prefix of counts (offsets[E_tot] = R)
      perm[r]          flat assignment id held by routed row r (rows sorted by expert, stable)
      inv_perm[f]      routed row of flat assignment f
      tiles[e]         ceil(M_e / tile_m)  (0 for an empty expert)
      tile_offsets[e]  exclusive prefix of tiles (tile_offsets[E_tot] = S)
      S                sum_e ceil(M_e / tile_m)                      (Eq. 16)
      mtile_expert / mtile_first_row / mtile_valid [S]  the m-tile table
      pad_row[f]       row of assignment f in the tile-padded layout in which expert e
                       starts at row tile_m * tile_offsets[e]
    Raises ValueError for an expert id outside [0, E_tot) or an expert repeated inside
    one token.
    """
    idx = np.asarray(topk_idx)
    if idx.ndim != 2:
        raise ValueError("topk_idx must be [T, k_tot]")
    T, k_tot = int(idx.shape[0]), int(idx.shape[1])
    R = T * k_tot
    flat = [int(v) for v in idx.reshape(-1)]

    # step 1: validate
    for t in range(T):
        seen = set()
        for j in range(k_tot):
            e = flat[t * k_tot + j]
            if e < 0 or e >= E_tot:
                raise ValueError(f"expert id {e} out of range at token {t}, slot {j}")
            if e in seen:
                raise ValueError(f"expert {e} repeated inside token {t}")
            seen.add(e)

    # step 2: counts and exclusive offsets
    counts = [0] * E_tot
    for e in flat:
        counts[e] += 1
    offsets = [0] * (E_tot + 1)
    for e in range(E_tot):
        offsets[e + 1] = offsets[e] + counts[e]
    assert offsets[E_tot] == R

    # step 3: stable counting sort of the flat assignment ids by expert
    seen_cnt = [0] * E_tot
    perm = [0] * R
    inv_perm = [0] * R
    for f in range(R):
        e = flat[f]
        r = offsets[e] + seen_cnt[e]
        seen_cnt[e] += 1
        perm[r] = f
        inv_perm[f] = r

    # step 4: tiles per expert, their prefix, the padded rows
    tiles = [ceil_div(counts[e], tile_m) for e in range(E_tot)]
    tile_offsets = [0] * (E_tot + 1)
    for e in range(E_tot):
        tile_offsets[e + 1] = tile_offsets[e] + tiles[e]
    S = tile_offsets[E_tot]
    pad_row = [0] * R
    for f in range(R):
        e = flat[f]
        pad_row[f] = tile_m * tile_offsets[e] + (inv_perm[f] - offsets[e])

    # step 5: the m-tile table
    mtile_expert = [0] * S
    mtile_first_row = [0] * S
    mtile_valid = [0] * S
    for e in range(E_tot):
        for i in range(tiles[e]):
            mu = tile_offsets[e] + i
            mtile_expert[mu] = e
            mtile_first_row[mu] = offsets[e] + i * tile_m
            mtile_valid[mu] = min(tile_m, counts[e] - i * tile_m)

    as32 = lambda a: np.asarray(a, dtype=np.int32)
    return dict(
        counts=as32(counts), offsets=as32(offsets), perm=as32(perm), inv_perm=as32(inv_perm),
        tiles=as32(tiles), tile_offsets=as32(tile_offsets), S=int(S),
        mtile_expert=as32(mtile_expert), mtile_first_row=as32(mtile_first_row),
        mtile_valid=as32(mtile_valid), pad_row=as32(pad_row),
    )


def brute_force_row(topk_idx, f: int) -> int:
    """Routed row of flat assignment f straight from the definition of a stable sort by
    expert: (# assignments of a smaller expert) + (# earlier assignments of the same one).
    O(R) per query; used as a pin on tiny inputs."""
    flat = [int(v) for v in np.asarray(topk_idx).reshape(-1)]
    e = flat[f]
    smaller = sum(1 for v in flat if v < e)
    earlier = sum(1 for g in range(f) if flat[g] == e)
    return smaller + earlier
