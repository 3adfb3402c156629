"""Seeded synthetic inputs for the MoE GEMM2 + GatherRS path.

This module only *makes inputs* (router decisions, activations, weights); none of the
operator's arithmetic lives here, so the CUDA path's tests, the CPU checker's tests and the
benchmark can all draw their data from it.

The paper replays router traces of trained models on a chat dataset (Section IV-A,
"Models and Workloads"); neither the models nor the traces are available, so routing is
synthetic with the same shapes and the same load-imbalance statistic
R_expert = max_e L_e / (M k / E):

* uniform   : logits iid U[0, 1) -> every expert equally likely;
* zipf      : logit[t, e] = sigma * z[t, e] + b_e,  z ~ N(0, 1),
              b_e = -s * ln(rank_e) with rank a seeded random permutation of 1..E;
              sigma is found by bisection on [0.25, 8] so that R_expert hits a target.
Top-k = the k largest logits (ties: lower expert id first), in descending order; the k
weights are the softmax of the selected logits (fp32, sum to 1).  "Shared" experts are extra
experts E, E+1, ... that every token is sent to with weight exactly 1.
Activations and weights are N(0, 0.02) rounded to bf16 (nearest even).
"""

from __future__ import annotations

import functools
from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    T: int                 # tokens
    H: int                 # hidden size (GEMM2 output width, the paper's N)
    I: int                 # expert intermediate size (full contraction length)
    E: int                 # routed experts
    k: int                 # routed experts per token
    n_shared: int = 0      # always-active shared experts
    TP: int = 1            # emulated tensor-parallel shards (split-K partials)
    EP: int = 1            # emulated destination ranks (output buffers)
    tile_m: int = 128
    tile_n: int = 128
    L: int = 1             # pipeline splits along H
    routing: str = "uniform"   # "uniform" | "zipf"
    zipf_s: float = 0.0
    target_r_expert: float = 0.0   # 0 = do not calibrate (sigma = sigma_fixed)
    sigma_fixed: float = 1.0
    routing_seed: int = 0
    data_seed: int = 1

    @property
    def k_tot(self) -> int:
        return self.k + self.n_shared

    @property
    def E_tot(self) -> int:
        return self.E + self.n_shared

    @property
    def R(self) -> int:
        return self.T * self.k_tot

    @property
    def K(self) -> int:
        return self.I // self.TP


TINY = Workload("tiny", T=256, H=256, I=128, E=8, k=2, TP=1, EP=2, tile_m=64, tile_n=64, L=1,
                routing="uniform", routing_seed=0, data_seed=1)
GRANITE = Workload("granite3moe", T=4096, H=1536, I=512, E=40, k=8, TP=2, EP=2,
                   tile_m=128, tile_n=256, L=1, routing="zipf", zipf_s=1.0,
                   target_r_expert=2.5, routing_seed=0, data_seed=1)
QWEN = Workload("qwen15moe", T=8192, H=2048, I=1408, E=60, k=4, TP=2, EP=2,
                tile_m=256, tile_n=256, L=1, routing="zipf", zipf_s=1.0,
                target_r_expert=2.5, routing_seed=0, data_seed=1)
DSV2L = Workload("dsv2lite", T=16384, H=2048, I=1408, E=64, k=6, n_shared=2, TP=2, EP=2,
                 tile_m=256, tile_n=256, L=2, routing="zipf", zipf_s=1.2,
                 target_r_expert=3.0, routing_seed=0, data_seed=1)

CONFIGS = {w.name: w for w in (TINY, GRANITE, QWEN, DSV2L)}


def sweep_workloads(T_list=(1024, 2048, 4096, 8192, 16384, 32768), s_list=(0.0, 0.6, 1.2),
                    EP_list=(1, 2, 4), tiles=((128, 128), (128, 256), (256, 256))):
    """The selector-regret sweep on the DeepSeek-V2-Lite shape."""
    out = []
    for iT, T in enumerate(T_list):
        for i_s, s in enumerate(s_list):
            for iEP, EP in enumerate(EP_list):
                for (tm, tn) in tiles:
                    out.append(replace(
                        DSV2L, name=f"sweep_T{T}_s{s}_EP{EP}_{tm}x{tn}", T=T, EP=EP,
                        tile_m=tm, tile_n=tn,
                        routing="uniform" if s == 0.0 else "zipf", zipf_s=s,
                        # s = 1.2 is calibrated to R_expert = 3; s = 0.6 reuses that sigma
                        target_r_expert=3.0 if s > 0.0 else 0.0,
                        routing_seed=1000 + 100 * iT + 10 * i_s + iEP))
    return out


# ----------------------------------------------------------------------------- routing

def _topk(logits: np.ndarray, k: int):
    order = np.argsort(-logits, axis=1, kind="stable")[:, :k]
    sel = np.take_along_axis(logits, order, axis=1).astype(np.float32)
    m = sel.max(axis=1, keepdims=True)
    p = np.exp(sel - m, dtype=np.float32)
    w = (p / p.sum(axis=1, keepdims=True, dtype=np.float32)).astype(np.float32)
    return order.astype(np.int32), w


def r_expert(idx_routed: np.ndarray, E: int) -> float:
    """max_e L_e / (M k / E) over the routed (non-shared) experts."""
    T, k = idx_routed.shape
    loads = np.bincount(idx_routed.reshape(-1), minlength=E)
    return float(loads.max() / (T * k / E))


def p90_load_ratio(idx_routed: np.ndarray, E: int) -> float:
    """90th percentile across experts of L_e / mean load."""
    T, k = idx_routed.shape
    loads = np.bincount(idx_routed.reshape(-1), minlength=E)
    return float(np.percentile(loads, 90) / (T * k / E))


@functools.lru_cache(maxsize=None)
def _zipf_parts(T: int, E: int, s: float, seed: int):
    rng = np.random.Generator(np.random.PCG64(seed))
    rank = rng.permutation(E) + 1
    bias = (-s * np.log(rank.astype(np.float64))).astype(np.float32)
    z = rng.standard_normal((T, E), dtype=np.float32)
    return bias, z


@functools.lru_cache(maxsize=None)
def calibrate_sigma(T: int, E: int, k: int, s: float, seed: int, target: float) -> float:
    """Bisection on sigma in [0.25, 8] (R_expert falls as the noise grows), 24 halvings."""
    bias, z = _zipf_parts(T, E, s, seed)
    lo, hi = 0.25, 8.0
    for _ in range(24):
        mid = 0.5 * (lo + hi)
        idx, _ = _topk(np.float32(mid) * z + bias, k)
        if r_expert(idx, E) > target:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def make_routing(w: Workload):
    """Returns (topk_idx int32 [T, k_tot], topk_w float32 [T, k_tot], info dict)."""
    if w.routing == "uniform":
        rng = np.random.Generator(np.random.PCG64(w.routing_seed))
        logits = rng.random((w.T, w.E), dtype=np.float32)
        sigma = None
    elif w.routing == "zipf":
        if w.target_r_expert > 0.0:
            # the sigma of the s = 1.2 calibration is reused for milder skews
            s_cal = w.zipf_s if w.zipf_s >= 1.0 else 1.2
            sigma = calibrate_sigma(w.T, w.E, w.k, s_cal, w.routing_seed, w.target_r_expert)
        else:
            sigma = w.sigma_fixed
        bias, z = _zipf_parts(w.T, w.E, w.zipf_s, w.routing_seed)
        logits = np.float32(sigma) * z + bias
    else:
        raise ValueError(w.routing)
    idx, wt = _topk(logits, w.k)
    info = dict(sigma=sigma, r_expert=r_expert(idx, w.E), p90_ratio=p90_load_ratio(idx, w.E))
    if w.n_shared:
        sh = np.broadcast_to(np.arange(w.E, w.E + w.n_shared, dtype=np.int32), (w.T, w.n_shared))
        idx = np.concatenate([idx, sh], axis=1)
        wt = np.concatenate([wt, np.ones((w.T, w.n_shared), dtype=np.float32)], axis=1)
    return np.ascontiguousarray(idx, dtype=np.int32), np.ascontiguousarray(wt, dtype=np.float32), info


# ----------------------------------------------------------------------------- data

def normal_bf16(shape, seed: int, std: float = 0.02) -> torch.Tensor:
    """N(0, std) in fp32 from a seeded CPU generator, rounded to bf16 (nearest even)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return (torch.randn(shape, generator=g, dtype=torch.float32) * std).to(torch.bfloat16)


def make_data(w: Workload):
    """x_routed bf16 [R, I] (rows iid: the operator's cost does not depend on values) and
    W2 bf16 [E_tot, H, I] (contraction index contiguous)."""
    x = normal_bf16((w.R, w.I), w.data_seed)
    W2 = normal_bf16((w.E_tot, w.H, w.I), w.data_seed + 7919)
    return x, W2


def make_gemm1_data(w: Workload):
    """Inputs of the up-stream stage: hidden states [T, H] ~ N(0, 1) (a normalised residual stream) and the
    gate/up weights W1 [E_tot, 2, I, H] ~ N(0, 0.02), bf16, from the data seed."""
    hidden = normal_bf16((w.T, w.H), w.data_seed + 101, std=1.0)
    W1 = normal_bf16((w.E_tot, 2, w.I, w.H), w.data_seed + 102, std=0.02)
    return hidden, W1


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (CPU) -> numpy uint16 view of its bit patterns."""
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
