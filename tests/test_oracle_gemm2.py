"""Pins for the GEMM2 + combine reference (plain C loops).

Each test checks the loops against something they do not contain: a dense masked
definition written with float64 matmuls, a library GEMM in the single-expert special case,
exactly representable identities, linearity, and invariance to how tokens are grouped.
"""

import numpy as np
import pytest
import torch

from oracle import gemm2_combine_ref as ref
from oracle import routing_ref as rr
from paper_2609_07536_b200 import workloads as wl


def _bits(a):
    """float array -> bf16 bit patterns (via torch's round-to-nearest-even)."""
    return wl.bf16_bits(torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def _tiny_problem(seed=0, T=40, E_tot=6, k_tot=3, H=24, I=40):
    rng = np.random.default_rng(seed)
    idx = np.stack([rng.permutation(E_tot)[:k_tot] for _ in range(T)]).astype(np.int32)
    w = rng.random((T, k_tot), dtype=np.float32)
    w /= w.sum(axis=1, keepdims=True)
    X_dense = _bits(rng.normal(0, 0.5, (T, E_tot, I)))
    W2 = _bits(rng.normal(0, 0.5, (E_tot, H, I)))
    r = rr.build_routing(idx, E_tot, 4)
    x_routed = np.zeros((T * k_tot, I), dtype=np.uint16)
    for t in range(T):
        for j in range(k_tot):
            x_routed[r["inv_perm"][t * k_tot + j]] = X_dense[t, idx[t, j]]
    return idx, w, X_dense, W2, r, x_routed


def test_matches_dense_masked_reference():
    idx, w, X_dense, W2, r, x_routed = _tiny_problem()
    dense = ref.dense_masked(X_dense, W2, idx, w)
    out64 = ref.gemm2_combine(x_routed, W2, idx, w, r["inv_perm"], accumulate="f64")
    out32 = ref.gemm2_combine(x_routed, W2, idx, w, r["inv_perm"], accumulate="f32")
    assert np.max(np.abs(out64 - dense)) < 1e-12
    assert np.max(np.abs(out32 - dense)) < 1e-5
    # a wrong expert, a wrong row or a dropped weight would be O(1) here
    assert np.max(np.abs(dense)) > 0.5


def test_tiny_config_f32_vs_f64_and_dense():
    w_ = wl.TINY
    idx, wt, _ = wl.make_routing(w_)
    r = rr.build_routing(idx, w_.E_tot, w_.tile_m)
    X_dense = wl.bf16_bits(wl.normal_bf16((w_.T, w_.E_tot, w_.I), 11))
    W2 = wl.bf16_bits(wl.normal_bf16((w_.E_tot, w_.H, w_.I), 12))
    x_routed = np.zeros((w_.R, w_.I), dtype=np.uint16)
    for t in range(w_.T):
        for j in range(w_.k_tot):
            x_routed[r["inv_perm"][t * w_.k_tot + j]] = X_dense[t, idx[t, j]]
    o32 = ref.gemm2_combine(x_routed, W2, idx, wt, r["inv_perm"])
    o64 = ref.gemm2_combine(x_routed, W2, idx, wt, r["inv_perm"], accumulate="f64")
    dense = ref.dense_masked(X_dense, W2, idx, wt)
    assert np.max(np.abs(o32 - o64)) < 1e-6      # the reference's own fp32 rounding
    assert np.max(np.abs(o64 - dense)) < 1e-12


def test_single_expert_is_a_plain_gemm():
    # E = 1, k = 1, w = 1  ->  out = x @ W2[0].T ; compare with a library matmul
    rng = np.random.default_rng(3)
    T, H, I = 50, 33, 72
    x = _bits(rng.normal(0, 1, (T, I)))
    W2 = _bits(rng.normal(0, 1, (1, H, I)))
    idx = np.zeros((T, 1), dtype=np.int32)
    w = np.ones((T, 1), dtype=np.float32)
    inv = np.arange(T, dtype=np.int32)
    out = ref.gemm2_combine(x, W2, idx, w, inv, accumulate="f64")
    lib = ref.bits_to_f64(x) @ ref.bits_to_f64(W2[0]).T
    assert np.max(np.abs(out - lib)) < 1e-11
    # transposed-operand mistake would change the shape or the values: H != I on purpose
    out32 = ref.gemm2_combine(x, W2, idx, w, inv)
    assert out32.shape == (T, H)
    assert np.max(np.abs(out32 - lib)) < 1e-4


def test_identity_weights_check_the_gather_exactly():
    # W2_e = identity (I = H): out[t] = sum_j w_j * x_routed[inv_perm[t, j]], and with
    # power-of-two weights and small integer x every value is exactly representable
    rng = np.random.default_rng(4)
    T, E, k, H = 30, 5, 2, 16
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    w = np.tile(np.array([0.5, 0.25], dtype=np.float32), (T, 1))
    r = rr.build_routing(idx, E, 4)
    xv = rng.integers(-8, 9, (T * k, H)).astype(np.float32)
    W2 = _bits(np.tile(np.eye(H, dtype=np.float32), (E, 1, 1)))
    out = ref.gemm2_combine(_bits(xv), W2, idx, w, r["inv_perm"])
    inv = r["inv_perm"].reshape(T, k)
    expect = 0.5 * xv[inv[:, 0]] + 0.25 * xv[inv[:, 1]]
    assert np.array_equal(out, expect)


def test_one_hot_rows_select_weight_columns():
    # x row = unit vector i0  ->  contribution = W2[e][:, i0]
    rng = np.random.default_rng(5)
    T, E, H, I = 12, 4, 10, 20
    idx = rng.integers(0, E, (T, 1)).astype(np.int32)
    w = np.ones((T, 1), dtype=np.float32)
    r = rr.build_routing(idx, E, 4)
    W2f = rng.integers(-5, 6, (E, H, I)).astype(np.float32)
    i0 = rng.integers(0, I, T)
    xv = np.zeros((T, I), dtype=np.float32)
    for t in range(T):
        xv[r["inv_perm"][t], i0[t]] = 1.0
    out = ref.gemm2_combine(_bits(xv), _bits(W2f), idx, w, r["inv_perm"])
    for t in range(T):
        assert np.array_equal(out[t], W2f[idx[t, 0], :, i0[t]])


def test_linearity_and_slot_order():
    idx, w, X_dense, W2, r, x_routed = _tiny_problem(seed=7)
    base = ref.gemm2_combine(x_routed, W2, idx, w, r["inv_perm"], accumulate="f64")
    doubled = ref.gemm2_combine(x_routed, W2, idx, 2 * w, r["inv_perm"], accumulate="f64")
    assert np.max(np.abs(doubled - 2 * base)) < 1e-12
    # swapping a token's slots (and their rows and weights with them) changes nothing
    T, k = idx.shape
    idx2, w2 = idx[:, ::-1].copy(), w[:, ::-1].copy()
    inv2 = r["inv_perm"].reshape(T, k)[:, ::-1].copy().reshape(-1)
    swapped = ref.gemm2_combine(x_routed, W2, idx2, w2, inv2, accumulate="f64")
    assert np.max(np.abs(swapped - base)) < 1e-12


def test_equal_experts_and_equal_rows_reduce_to_one_gemm():
    # all W2_e equal, all rows of a token equal, weights sum to 1  ->  out[t] = x_t @ W2.T
    rng = np.random.default_rng(8)
    T, E, k, H, I = 20, 4, 3, 8, 16
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    w = rng.random((T, k), dtype=np.float32)
    w /= w.sum(axis=1, keepdims=True)
    r = rr.build_routing(idx, E, 4)
    xt = _bits(rng.normal(0, 1, (T, I)))
    x_routed = np.zeros((T * k, I), dtype=np.uint16)
    for t in range(T):
        for j in range(k):
            x_routed[r["inv_perm"][t * k + j]] = xt[t]
    W1 = _bits(rng.normal(0, 1, (1, H, I)))
    out = ref.gemm2_combine(x_routed, np.tile(W1, (E, 1, 1)), idx, w, r["inv_perm"], accumulate="f64")
    expect = ref.bits_to_f64(xt) @ ref.bits_to_f64(W1[0]).T * w.astype(np.float64).sum(axis=1, keepdims=True)
    assert np.max(np.abs(out - expect)) < 1e-11


def test_token_subset_and_rank_split():
    idx, w, X_dense, W2, r, x_routed = _tiny_problem(seed=9)
    full = ref.gemm2_combine(x_routed, W2, idx, w, r["inv_perm"])
    toks = np.array([39, 0, 17, 17, 5], dtype=np.int32)
    sub = ref.gemm2_combine(x_routed, W2, idx, w, r["inv_perm"], tokens=toks)
    assert np.array_equal(sub, full[toks])
    for EP in (1, 2, 3, 4, 7):
        parts = ref.split_by_rank(full, EP)
        assert len(parts) == EP
        assert np.array_equal(np.concatenate(parts), full)
        blk = -(-full.shape[0] // EP)
        assert all(p.shape[0] <= blk for p in parts)
    with pytest.raises(ValueError):
        ref.gemm2_combine(x_routed, W2, idx, w, r["inv_perm"], tokens=np.array([40], dtype=np.int32))


def test_round_bf16_matches_torch():
    rng = np.random.default_rng(10)
    a = rng.normal(0, 1, 4096).astype(np.float32)
    a[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]     # ties: to even
    assert np.array_equal(ref.round_bf16(a), _bits(a))
