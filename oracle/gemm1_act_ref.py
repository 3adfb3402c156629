"""Python face of the GEMM1 + gated-activation reference (CPU oracle, test infrastructure).

Only the tests and the benchmark's CPU legs may import this file.

* gemm1_act()   calls the plain C loops of gemm1_act_ref.c (fp32 or fp64): routed row r of x_routed
                belongs to assignment perm[r] = t * k_tot + j, expert topk_idx[t][j]
                (Section II-A, steps 1-2; SiLU gating is the reading taken for "a gated activation").
* dense_f64()   the same definition written with numpy float64 matmuls, expert by expert; it pins the
                C loops against a second, differently written definition.

hidden [T, H] and W1 [E_tot, 2, I, H] (plane 0 gate, plane 1 up) are bf16 bit patterns (numpy uint16).
"""

from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        u16p = ctypes.POINTER(ctypes.c_uint16)
        common = [u16p, u16p, i32p, i32p] + [ctypes.c_int] * 5 + [i32p, ctypes.c_int]
        lib.moe_ref_gemm1_act_f32.argtypes = common + [ctypes.POINTER(ctypes.c_float)]
        lib.moe_ref_gemm1_act_f32.restype = ctypes.c_int
        lib.moe_ref_gemm1_act_f64.argtypes = common + [ctypes.POINTER(ctypes.c_double)]
        lib.moe_ref_gemm1_act_f64.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def gemm1_act(hidden_bits, W1_bits, topk_idx, perm, rows=None, f64: bool = False) -> np.ndarray:
    """x_routed rows (unrounded), [n_rows, I]; rows = None evaluates every routed row."""
    hidden_bits = np.ascontiguousarray(hidden_bits, dtype=np.uint16)
    W1_bits = np.ascontiguousarray(W1_bits, dtype=np.uint16)
    topk_idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    T, H = hidden_bits.shape
    E_tot, two, I, H2 = W1_bits.shape
    assert two == 2 and H2 == H and topk_idx.shape[0] == T
    k_tot = topk_idx.shape[1]
    assert perm.shape == (T * k_tot,)
    if rows is None:
        n, rp = T * k_tot, None
    else:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        n, rp = len(rows), _ptr(rows, ctypes.c_int32)
    out = np.empty((n, I), dtype=np.float64 if f64 else np.float32)
    fn = _load().moe_ref_gemm1_act_f64 if f64 else _load().moe_ref_gemm1_act_f32
    rc = fn(_ptr(hidden_bits, ctypes.c_uint16), _ptr(W1_bits, ctypes.c_uint16), _ptr(topk_idx, ctypes.c_int32),
            _ptr(perm, ctypes.c_int32), T, H, I, E_tot, k_tot, rp, n,
            _ptr(out, ctypes.c_double if f64 else ctypes.c_float))
    if rc != 0:
        raise ValueError("index out of range in the GEMM1 reference")
    return out


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def dense_f64(hidden_bits, W1_bits, topk_idx, perm) -> np.ndarray:
    """The definition with float64 matmuls: every token through the gate and up matrices of each of its
    experts, then silu(gate) * up; rows placed by perm."""
    h = bits_to_f64(hidden_bits)
    W = bits_to_f64(W1_bits)
    T, k_tot = topk_idx.shape
    I = W.shape[2]
    x = np.zeros((T * k_tot, I))
    inv = np.empty(T * k_tot, dtype=np.int64)
    inv[np.asarray(perm, dtype=np.int64)] = np.arange(T * k_tot)
    for e in range(W.shape[0]):
        ts, js = np.nonzero(topk_idx == e)
        if len(ts) == 0:
            continue
        g = h[ts] @ W[e, 0].T
        u = h[ts] @ W[e, 1].T
        x[inv[ts * k_tot + js]] = g / (1.0 + np.exp(-g)) * u
    return x
