"""Pins of the GEMM1 + gated-activation reference (CPU only): a second definition in float64
matmuls, closed forms of the activation, the row -> (token, expert) mapping by brute force."""

import math

import numpy as np
import torch

from oracle import gemm1_act_ref as g1
from oracle import routing_ref as rr
from paper_2609_07536_b200 import workloads as wl


def _bits(a: np.ndarray) -> np.ndarray:
    return wl.bf16_bits(torch.from_numpy(np.asarray(a, dtype=np.float32)).bfloat16())


def _case(T=40, H=48, I=24, E=5, k=2, seed=0, scale_h=1.0):
    rng = np.random.default_rng(seed)
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    hidden = _bits(rng.standard_normal((T, H)) * scale_h)
    W1 = _bits(rng.standard_normal((E, 2, I, H)) * 0.2)
    r = rr.build_routing(idx, E, 64)
    return hidden, W1, idx, r["perm"]


def test_against_the_float64_matmul_definition():
    hidden, W1, idx, perm = _case()
    ref = g1.dense_f64(hidden, W1, idx, perm)
    got64 = g1.gemm1_act(hidden, W1, idx, perm, f64=True)
    got32 = g1.gemm1_act(hidden, W1, idx, perm)
    assert np.max(np.abs(got64 - ref)) < 1e-12
    assert np.max(np.abs(got32 - ref)) < 2e-5 * max(1.0, np.max(np.abs(ref)))
    # a subset of rows gives the same rows
    rows = np.array([3, 0, 17, 79], dtype=np.int32)
    assert np.array_equal(g1.gemm1_act(hidden, W1, idx, perm, rows=rows), got32[rows])


def test_row_belongs_to_the_token_and_expert_of_its_assignment():
    # brute force, one scalar at a time, straight from the definition
    hidden, W1, idx, perm = _case(T=7, H=8, I=3, E=4, k=2, seed=3)
    h, W = g1.bits_to_f64(hidden), g1.bits_to_f64(W1)
    got = g1.gemm1_act(hidden, W1, idx, perm, f64=True)
    for r in range(len(perm)):
        t, j = divmod(int(perm[r]), 2)
        e = int(idx[t, j])
        for i in range(3):
            g = sum(h[t, c] * W[e, 0, i, c] for c in range(8))
            u = sum(h[t, c] * W[e, 1, i, c] for c in range(8))
            assert abs(got[r, i] - g / (1.0 + math.exp(-g)) * u) < 1e-12


def test_activation_closed_forms():
    # one token, one expert, one-hot hidden row: g = Wg[i][0], u = Wu[i][0] exactly
    T, H, I = 1, 4, 6
    idx = np.zeros((1, 1), dtype=np.int32)
    perm = np.zeros(1, dtype=np.int32)
    hidden = _bits(np.array([[1.0, 0.0, 0.0, 0.0]]))
    gates = np.array([0.0, 1.0, -1.0, 32.0, -32.0, 2.0])
    ups = np.array([3.0, 1.0, 1.0, 0.5, 1.0, -1.5])
    W = np.zeros((1, 2, I, H), dtype=np.float32)
    W[0, 0, :, 0], W[0, 1, :, 0] = gates, ups
    out = g1.gemm1_act(hidden, _bits(W), idx, perm, f64=True)[0]
    assert out[0] == 0.0                                     # silu(0) = 0
    assert abs(out[1] - 0.7310585786300049) < 1e-15          # silu(1) = 1 / (1 + 1/e)
    assert abs(out[2] + 0.2689414213699951) < 1e-15          # silu(-1) = -1 / (1 + e)
    assert out[3] == 32.0 / (1.0 + math.exp(-32.0)) * 0.5    # ~ 16: silu(z) -> z for large z
    assert abs(out[3] - 16.0) < 1e-12
    assert abs(out[4]) < 1e-12                               # silu(z) -> 0 for very negative z
    assert abs(out[5] - 2.0 / (1.0 + math.exp(-2.0)) * -1.5) < 1e-15
    out32 = g1.gemm1_act(hidden, _bits(W), idx, perm)[0]
    assert out32[0] == 0.0 and out32[3] == 16.0              # exact in fp32 too
    assert np.max(np.abs(out32 - out)) < 1e-6


def test_gate_symmetry_and_linearity_in_the_up_path():
    hidden, W1, idx, perm = _case(seed=5)
    Wf = g1.bits_to_f64(W1).astype(np.float32)
    neg = Wf.copy()
    neg[:, 0] *= -1.0                                        # negate every gate weight (exact in bf16)
    a = g1.gemm1_act(hidden, W1, idx, perm, f64=True)
    b = g1.gemm1_act(hidden, _bits(neg), idx, perm, f64=True)
    # silu(z) - silu(-z) = z: with a = silu(g) u and b = silu(-g) u, a - b = g u
    h, W = g1.bits_to_f64(hidden), g1.bits_to_f64(W1)
    inv = np.empty(len(perm), dtype=np.int64)
    inv[perm] = np.arange(len(perm))
    for t in range(0, hidden.shape[0], 7):
        for j in range(idx.shape[1]):
            e, r = int(idx[t, j]), int(inv[t * idx.shape[1] + j])
            g, u = W[e, 0] @ h[t], W[e, 1] @ h[t]
            assert np.max(np.abs((a[r] - b[r]) - g * u)) < 1e-12
    # doubling the up weights doubles the result exactly (power of two)
    dbl = Wf.copy()
    dbl[:, 1] *= 2.0
    c = g1.gemm1_act(hidden, _bits(dbl), idx, perm)
    assert np.array_equal(c, 2.0 * g1.gemm1_act(hidden, W1, idx, perm))
    # zero gate weights: silu(0) * u = 0 everywhere
    zg = Wf.copy()
    zg[:, 0] = 0.0
    assert not g1.gemm1_act(hidden, _bits(zg), idx, perm).any()
