"""Python face of the GEMM2 + combine reference (CPU oracle, test infrastructure).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this file.

* gemm2_combine()     calls the plain C loops of gemm2_combine_ref.c (fp32 or fp64 sums);
* split_by_rank()     hands each destination rank its contiguous block of tokens
                      (rank d owns tokens [d*ceil(T/EP), (d+1)*ceil(T/EP)) -- Section III-C:
                      every rank ends up owning about ceil(M/D) original tokens);
* dense_masked()      the "every token through every expert, unselected ones masked"
                      definition on tiny inputs, written with numpy float64 matmuls; it pins
                      the C loops against a second, differently written definition.

Inputs are bf16 bit patterns carried as numpy uint16 arrays.
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
        f32p = ctypes.POINTER(ctypes.c_float)
        f64p = ctypes.POINTER(ctypes.c_double)
        common = [u16p, u16p, i32p, f32p, i32p] + [ctypes.c_int] * 5 + [i32p, ctypes.c_int]
        lib.moe_ref_gemm2_combine_f32.argtypes = common + [f32p]
        lib.moe_ref_gemm2_combine_f32.restype = ctypes.c_int
        lib.moe_ref_gemm2_combine_f64.argtypes = common + [f64p]
        lib.moe_ref_gemm2_combine_f64.restype = ctypes.c_int
        lib.moe_ref_round_bf16.argtypes = [f32p, u16p, ctypes.c_long]
        lib.moe_ref_round_bf16.restype = None
        lib.moe_ref_threads.argtypes = []
        lib.moe_ref_threads.restype = ctypes.c_int
        lib.moe_ref_set_threads.argtypes = [ctypes.c_int]
        lib.moe_ref_set_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Threads the C loops will use (OpenMP's maximum)."""
    return int(_load().moe_ref_threads())


def set_threads(n: int) -> int:
    """Limits the C loops to n threads; returns the previous maximum (to restore it)."""
    return int(_load().moe_ref_set_threads(int(n)))


def _ptr(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def gemm2_combine(x_routed_bits, W2_bits, topk_idx, topk_w, inv_perm, tokens=None,
                  accumulate: str = "f32") -> np.ndarray:
    """out[r, :] for the listed tokens (all tokens when `tokens` is None).

    x_routed_bits uint16 [R, I]; W2_bits uint16 [E_tot, H, I]; topk_idx int32 [T, k_tot];
    topk_w float32 [T, k_tot]; inv_perm int32 [T*k_tot].  Returns float32 (or float64 when
    accumulate == "f64") of shape [n_tokens, H]."""
    lib = _load()
    x = np.ascontiguousarray(x_routed_bits, dtype=np.uint16)
    W = np.ascontiguousarray(W2_bits, dtype=np.uint16)
    idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    w = np.ascontiguousarray(topk_w, dtype=np.float32)
    inv = np.ascontiguousarray(inv_perm, dtype=np.int32).reshape(-1)
    T, k_tot = idx.shape
    E_tot, H, I = W.shape
    assert x.shape == (T * k_tot, I) and w.shape == (T, k_tot) and inv.shape == (T * k_tot,)
    if tokens is None:
        n = T
        tok_ptr = ctypes.POINTER(ctypes.c_int32)()
    else:
        tok = np.ascontiguousarray(tokens, dtype=np.int32).reshape(-1)
        n = int(tok.shape[0])
        tok_ptr = _ptr(tok, ctypes.c_int32)
    args = [_ptr(x, ctypes.c_uint16), _ptr(W, ctypes.c_uint16), _ptr(idx, ctypes.c_int32),
            _ptr(w, ctypes.c_float), _ptr(inv, ctypes.c_int32), T, H, I, E_tot, k_tot, tok_ptr, n]
    if accumulate == "f32":
        out = np.empty((n, H), dtype=np.float32)
        rc = lib.moe_ref_gemm2_combine_f32(*args, _ptr(out, ctypes.c_float))
    elif accumulate == "f64":
        out = np.empty((n, H), dtype=np.float64)
        rc = lib.moe_ref_gemm2_combine_f64(*args, _ptr(out, ctypes.c_double))
    else:
        raise ValueError(accumulate)
    if rc != 0:
        raise ValueError("index out of range in the routing arrays")
    return out


def round_bf16(a) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().moe_ref_round_bf16(_ptr(a, ctypes.c_float), _ptr(out, ctypes.c_uint16), a.size)
    return out


def bits_to_f64(bits) -> np.ndarray:
    """bf16 bit patterns -> float64 values (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def split_by_rank(out_tokens: np.ndarray, EP: int) -> list:
    """Token-ordered [T, H] -> list of EP arrays, rank d holding its block of
    ceil(T/EP) tokens (the last ranks may hold fewer, or none)."""
    T = out_tokens.shape[0]
    blk = -(-T // EP)
    return [out_tokens[min(T, d * blk):min(T, (d + 1) * blk)] for d in range(EP)]


def dense_masked(X_dense_bits, W2_bits, topk_idx, topk_w) -> np.ndarray:
    """out[t] = sum_e gate[t, e] * (X_dense[t, e, :] @ W2[e].T), gate[t, e] = the weight of
    expert e for token t if it was selected, else 0.  X_dense_bits uint16 [T, E_tot, I]
    holds an input row for *every* (token, expert) pair; the routed path only ever sees the
    selected ones.  float64 throughout."""
    X = bits_to_f64(X_dense_bits)
    W = bits_to_f64(W2_bits)
    idx = np.asarray(topk_idx)
    w = np.asarray(topk_w, dtype=np.float64)
    T, E_tot, I = X.shape
    H = W.shape[1]
    gate = np.zeros((T, E_tot), dtype=np.float64)
    for t in range(T):
        for j in range(idx.shape[1]):
            gate[t, int(idx[t, j])] = w[t, j]
    out = np.zeros((T, H), dtype=np.float64)
    for e in range(E_tot):
        y_e = X[:, e, :] @ W[e].T          # every token through expert e
        out += gate[:, e:e + 1] * y_e      # unselected tokens are masked by a zero gate
    return out
