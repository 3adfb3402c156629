"""Benchmark of the MoE GEMM2 + GatherRS hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload dsv2lite] [--impl reference]
    python bench.py --sweep [--sweep-out sweep.json]                 (selector-regret sweep)

One step = one pass of the whole hot path over one batch: routing/tile-count build (GPU) ->
tile counts to the host -> analytical plan (host) -> fused grouped GEMM2 + combine (GPU).
Prints ONE JSON line.  `value` is microseconds per layer (lower is better) with the inputs
resident in HBM; `e2e` is the same through the host-buffer entry point with host<->device
copies inside the timed region; `roofline` describes the fused kernel; `cpu_baseline` is the
CPU oracle timed on this machine's host cores on a bounded token sample.

With N > 1 (torchrun) every rank runs an independent replica (the operator is single-GPU by
construction: no data-path collective); NCCL is used only for the barrier and the max.
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused GEMM2+combine us/layer (whole step: routing build + analytical plan + fused kernel)"
# workload -> (dram__bytes_read.sum + dram__bytes_write.sum of one fused launch, (tile_m, tile_n, L, co_warps) it was captured at)
NCU_TRAFFIC_BYTES = {"dsv2lite": (1785131264 + 1096537344, (256, 256, 2, 0))}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def config_of(w, info, world):
    """The `config` object of the JSON line: the same dict in the main arm and in the reference arm."""
    x_mb, w2_mb = w.R * w.I * 2 / 1e6, w.E_tot * w.H * w.I * 2 / 1e6
    y_mb = w.T * w.L * w.k_tot * w.TP * (-(-w.H // w.L)) * 2 / 1e6
    return {"workload": w.name, "T": w.T, "H": w.H, "I": w.I, "E": w.E, "k": w.k,
            "n_shared": w.n_shared, "TP": w.TP, "EP": w.EP, "tile": f"{w.tile_m}x{w.tile_n}",
            "L": w.L, "routing": f"{w.routing} s={w.zipf_s}", "r_expert": info["r_expert"],
            "p90_ratio": info["p90_ratio"],
            "l2": f"inputs larger than L2 (x {x_mb:.0f} MB, W2 {w2_mb:.0f} MB, Y {y_mb:.0f} MB vs 126 MB)"
                  if x_mb + w2_mb + y_mb > 252 else
                  f"inputs x {x_mb:.0f} MB, W2 {w2_mb:.0f} MB, Y {y_mb:.0f} MB; a 256 MB buffer is written between timed steps to flush L2",
            "replicas": "independent per GPU, no collective" if world > 1 else "single GPU"}


# ----------------------------------------------------------------------------- replicas

def max_over_ranks(values, world, device="cpu"):
    """Replicas only: every rank runs the same independent workload, the job's time is the slowest rank's.
    Works on any initialised process group (NCCL on the GPU machine, gloo in the CPU tests)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def job_value(us_per_layer_slowest_rank, world):
    """N independent replicas finish N layers in the time of the slowest one: us per layer of the whole job."""
    return us_per_layer_slowest_rank / max(1, world)


# ----------------------------------------------------------------------------- roofline denominator

def tensor_peak_for(peaks, loop_seconds, clocks):
    """Which measured cuBLAS figure a tensor-bound kernel is set against.  The burst figure (a kernel timed
    alone, clocks at their maximum) unless the timed loop itself lasted at least a second AND the SM clock
    sampled during it sat below 0.9 of its maximum (the power-capped steady state the sustained figure was
    measured in).  Returns (TFLOP/s, the rule spelled out with the run's own numbers)."""
    sust = peaks.get("bf16_tflops_sustained")
    mhz, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    capped = bool(sust) and loop_seconds >= 1.0 and mhz is not None and mx and mhz < 0.9 * mx
    why = (f"timed loop {loop_seconds:.3f} s, median SM clock {mhz} of {mx} MHz -> "
           + ("sustained figure (loop >= 1 s and clock < 0.9 max)" if capped else "burst figure (a loop shorter than 1 s, or a clock at >= 0.9 max)"))
    return (sust if capped else peaks["bf16_tflops"]), why


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
        except Exception as exc:  # NVML missing: report no clocks rather than fail the bench
            self.nv, self.err = None, repr(exc)

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- workload on the device

class DeviceWorkload:
    def __init__(self, w, device, data="seeded"):
        import numpy as np
        import torch
        from paper_2609_07536_b200 import binding as B
        from paper_2609_07536_b200 import workloads as wl
        self.w, self.B, self.torch = w, B, torch
        self.idx, self.wt, self.info = wl.make_routing(w)
        if data == "seeded":
            self.x_cpu, self.W2_cpu = wl.make_data(w)
            self.x, self.W2 = self.x_cpu.to(device), self.W2_cpu.to(device)
        else:  # values do not affect timing: draw them on the device
            g = torch.Generator(device=device).manual_seed(w.data_seed)
            self.x = (torch.randn((w.R, w.I), generator=g, device=device) * 0.02).bfloat16()
            self.W2 = (torch.randn((w.E_tot, w.H, w.I), generator=g, device=device) * 0.02).bfloat16()
        self.idx_d = torch.from_numpy(self.idx).to(device)
        self.wt_d = torch.from_numpy(self.wt).to(device)
        self.shape = B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
        self.ws = B.alloc_workspace(self.shape, w.tile_m, w.tile_n, device=device)
        self.flops = 2.0 * w.R * w.I * w.H
        self.combine_bytes = w.TP * w.R * w.H * 2 + w.T * w.H * 2 + w.R * 8


def make_stepper(h, dw, limits_override=None):
    """Returns step(...) -> (plan, counts): the whole hot path on device-resident inputs."""
    B, torch, w, ws = dw.B, dw.torch, dw.w, dw.ws
    occ, lim, rho = B.moe_query_occupancy(h, w.tile_m, w.tile_n)
    if limits_override:
        for k, v in limits_override.items():
            setattr(lim, k, v)
    stream = torch.cuda.current_stream()
    E = w.E_tot

    w_default = lim.force_co_warps

    def step(force_C=0, mode=B.MOE_MODE_FUSED, ev_before=None, ev_after=None, P_override=None,
             C_override=None, reuse=None, force_w=None):
        if reuse is None:
            B.moe_build_routing(h, dw.idx_d, dw.shape, w.tile_m, ws.routing, ws.tile_counts, ws.status)
            stream.synchronize()                               # tile counts are on the host now
            counts = ws.tile_counts[:E + 1].tolist()
        else:                                                  # sweeps: routing already built
            counts = reuse
        lim.force_comm_ctas = force_C
        lim.force_co_warps = w_default if force_w is None else force_w
        plan = B.plan_partition(counts[:E], occ, lim, dw.shape, rho)
        lim.force_co_warps = w_default
        plan.mode = mode
        if P_override is not None:
            plan.P = P_override
        if C_override is not None:
            plan.comm_ctas = plan.R = C_override
        if ev_before is not None:
            ev_before.record(stream)
        B.moe_gemm2_combine(h, dw.x, dw.W2, None, dw.wt_d, dw.shape, occ, ws.routing, counts[E], plan,
                            ws.out, ws.y_ws, ws.flags_ws, ws.status)
        if ev_after is not None:
            ev_after.record(stream)
        return plan, counts

    return step, (occ, lim, rho)


def time_fused(step, torch, force_C, n_warm, n_samples, **kw):
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_samples)]
    for _ in range(n_warm):
        step(force_C, **kw)
    for a, b in evs:
        step(force_C, ev_before=a, ev_after=b, **kw)
    torch.cuda.synchronize()
    return [a.elapsed_time(b) * 1e3 for a, b in evs]   # us


# ----------------------------------------------------------------------------- measured selection oracle
# Section IV-B: the measured oracle is the C with the lowest median latency over a sweep of every
# legal C; regret = (T_pick - T_best) / T_best.

def time_all_C(step, torch, counts, cands, n_warm=1, n_samples=5):
    """Median fused-kernel time [us] for every candidate (C, w) (routing is reused).  The candidates are
    interleaved: every round visits all of them in a fresh seeded random order, so that slow drifts
    of the GPU's state (power capping sets in after a second or two of load) hit every candidate alike."""
    import random
    rng = random.Random(1234)
    order = list(cands)
    for _ in range(n_warm):
        for C, w in order:
            step(C, reuse=counts, force_w=w)
    samples = {c: [] for c in order}
    evs = []
    for _ in range(n_samples):
        rng.shuffle(order)
        for C, w in order:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            step(C, ev_before=a, ev_after=b, reuse=counts, force_w=w)
            evs.append(((C, w), a, b))
    torch.cuda.synchronize()
    for c, a, b in evs:
        samples[c].append(a.elapsed_time(b) * 1e3)
    return {c: statistics.median(v) for c, v in samples.items()}


def regret_of_workload(step, torch, counts, lim, picked, n_warm=1, n_samples=5, C_hi=None, keep_curve=True):
    """Times every member of the legal set -- C in 1..C_max without co-resident warps and, where the kernel
    family has them (drain help), C in 1..C_co_max with w in 1..co_warps_max -- and compares the analytical
    pick `picked` = (C, w)."""
    C_hi = C_hi or lim.C_max
    cands = {(C, 0) for C in range(1, C_hi + 1)}
    if lim.drain_help and lim.co_warps_max > 0:
        cands |= {(C, w) for C in range(1, min(C_hi, lim.C_co_max) + 1) for w in range(1, lim.co_warps_max + 1)}
    cands.add(tuple(picked))
    times = time_all_C(step, torch, counts, sorted(cands), n_warm, n_samples)
    best = min(times, key=times.get)
    t_best, t_pick = times[best], times[tuple(picked)]
    out = {"picked_C": picked[0], "picked_w": picked[1], "t_pick_us": t_pick, "best_C": best[0], "best_w": best[1],
           "t_best_us": t_best, "regret": (t_pick - t_best) / t_best,
           "regret_static_C3": (times[(3, 0)] - t_best) / t_best if (3, 0) in times else None,
           "best_without_co_warps_us": min(t for (C, w), t in times.items() if w == 0),
           "swept_C": [1, C_hi], "candidates": len(times), "samples_per_C": n_samples}
    if keep_curve:
        out["times_us"] = {f"{c}" if w == 0 else f"{c}w{w}": round(t, 1) for (c, w), t in times.items()}
    return out


def run_sweep(h, args, peaks):
    """The regret sweep on the DeepSeek-V2-Lite shape: T x Zipf s x EP x tile, every legal C, for the
    paper's static partition (drain_help = 0) and for the default mode (drain_help = 1)."""
    import torch
    from paper_2609_07536_b200 import workloads as wl
    device = f"cuda:{torch.cuda.current_device()}"
    results = []
    for w in wl.sweep_workloads():
        if args.sweep_filter and args.sweep_filter not in w.name:
            continue
        dw = DeviceWorkload(w, device, data="device")
        row = dict(name=w.name, T=w.T, zipf_s=w.zipf_s, EP=w.EP, tile=f"{w.tile_m}x{w.tile_n}", L=w.L,
                   r_expert=dw.info["r_expert"])
        for dh in ((0,) if args.sweep_modes == "static" else (1,) if args.sweep_modes == "drain_help" else (0, 1)):
            step, (occ, lim, rho) = make_stepper(h, dw, limits_override=dict(drain_help=dh, dep_model=args.dep_model))
            plan, counts = step()
            torch.cuda.synchronize()
            r = regret_of_workload(step, torch, counts, lim, (plan.comm_ctas, plan.co_warps), n_warm=1,
                                   n_samples=args.sweep_samples * (2 if w.T <= 4096 else 1) + (1 if w.T <= 4096 else 0),
                                   keep_curve=args.sweep_curves)   # short launches are noisier: twice the samples
            r.update(W_comp=plan.W_comp, W_comm=plan.W_comm, rho=plan.rho_q / 2 ** 20,
                     roofline_frac=(dw.flops / peaks["bf16_tflops"] / 1e6) / r["t_pick_us"])
            row["static" if dh == 0 else "drain_help"] = r
        results.append(row)
        if "static" not in row or "drain_help" not in row:
            k = "static" if "static" in row else "drain_help"
            print(f"{w.name}: {k} pick C={row[k]['picked_C']} w={row[k]['picked_w']} {row[k]['t_pick_us']:.0f} us best C={row[k]['best_C']} "
                  f"w={row[k]['best_w']} {row[k]['t_best_us']:.0f} us regret {100 * row[k]['regret']:.1f}%", flush=True)
            del dw, step
            torch.cuda.empty_cache()
            continue
        a, b = row["static"], row["drain_help"]
        print(f"{w.name}: static pick C={a['picked_C']} {a['t_pick_us']:.0f} us best C={a['best_C']} {a['t_best_us']:.0f} us "
              f"regret {100 * a['regret']:.1f}% (C=3: {100 * a['regret_static_C3']:.0f}%) | drain-help pick C={b['picked_C']} "
              f"w={b['picked_w']} {b['t_pick_us']:.0f} us best C={b['best_C']} w={b['best_w']} {b['t_best_us']:.0f} us "
              f"regret {100 * b['regret']:.1f}%", flush=True)
        del dw, step
        torch.cuda.empty_cache()
    summary = {"n": len(results)}
    for key in ("static", "drain_help"):
        regs = [r[key]["regret"] for r in results if key in r]
        if regs:
            rows = [r[key] for r in results if key in r]
            summary[key] = {"mean_regret": statistics.mean(regs), "max_regret": max(regs),
                            "mean_regret_static_C3": statistics.mean(r["regret_static_C3"] for r in rows),
                            "geomean_speedup_pick_over_C3": statistics.geometric_mean(
                                (1 + r["regret_static_C3"]) / (1 + r["regret"]) for r in rows),
                            "picks_with_co_warps": sum(1 for r in rows if r["picked_w"] > 0),
                            "best_with_co_warps": sum(1 for r in rows if r["best_w"] > 0),
                            "geomean_best_over_best_without_co_warps": statistics.geometric_mean(
                                r["t_best_us"] / r["best_without_co_warps_us"] for r in rows)}
    os.makedirs(os.path.dirname(args.sweep_out) or ".", exist_ok=True)
    json.dump({"summary": summary, "results": results}, open(args.sweep_out, "w"))
    print(json.dumps({"sweep_summary": summary}))


def calibrate(h, device, C_ref=32, tile=(128, 256)):
    """Eq. 13 on this GPU: rho_ref = (time of one communication wave) / (time of one compute wave),
    both measured with the role running alone on its share of the SMs at a fixed C_ref, on the
    reference workload (DeepSeek-V2-Lite shape, T = 4096, uniform routing, 128x256, TP = EP = L = 2)."""
    import torch
    from dataclasses import replace
    from paper_2609_07536_b200 import binding as B
    from paper_2609_07536_b200 import workloads as wl
    w = replace(wl.DSV2L, name="rho_ref", T=4096, routing="uniform", zipf_s=0.0, target_r_expert=0.0,
                tile_m=tile[0], tile_n=tile[1])
    dw = DeviceWorkload(w, device, data="device")
    rho, wave_comp, wave_comm = B.moe_calibrate_rho(h, dw.x, dw.W2, dw.idx_d, dw.wt_d, dw.ws, C_ref=C_ref, n_samples=15)
    print(json.dumps({"calibration": {
        "workload": f"DeepSeek-V2-Lite shape, T=4096, uniform, {w.tile_m}x{w.tile_n}, TP=2, EP=2, L=2", "C_ref": C_ref,
        "us_per_compute_wave": wave_comp, "us_per_comm_wave": wave_comm,
        "rho_ref": rho.rho_ref, "K_ref": rho.K_ref, "tile_ref": [rho.tile_m_ref, rho.tile_n_ref],
        "rows_ref": rho.rows_ref, "comm_cols_ref": rho.comm_cols_ref, "D_ref": rho.D_ref}}))


# ----------------------------------------------------------------------------- other workloads, briefly

def all_traffic_bytes(w, x_passes=1):
    """Every byte one launch has to move through HBM: x (once per pass), W2, Y written and read back, out."""
    return (w.R * w.I * 2 * x_passes + w.E_tot * w.H * w.I * 2 +
            2 * w.T * w.L * w.k_tot * w.TP * (-(-w.H // w.L)) * 2 + w.T * w.H * 2)


def routing_launches(R):
    """Launches of one routing build: one (a single CTA, or a single cluster) up to 128 chunks of 256 assignments,
    four (histogram, column scan, finalize, scatter) beyond."""
    return 1 if (R + 255) // 256 <= 128 else 4


def quick_config(h, w, device, peaks, steps=30, warm=5, counts_on_device_too=False):
    """A bounded measurement of one more workload (a second or two): the whole step timed like the headline
    one (K moe_layer calls between two events), the fused kernel by events around its launch.  Fractions
    against the headline roofline (GEMM FLOPs at the burst peak -- these loops last milliseconds -- or combine
    bytes at the copy bandwidth, whichever is slower) and against the time all of the launch's HBM traffic needs."""
    import torch
    dw = DeviceWorkload(w, device, data="device")
    B = dw.B
    occ, lim, rho = B.moe_query_occupancy(h, w.tile_m, w.tile_n)
    layer = B.LayerCall(h, dw.x, dw.W2, dw.idx_d, dw.wt_d, dw.ws, limits=lim)
    for _ in range(warm):
        plan = layer()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record(); b.record()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for a, b in evs:
        plan = layer(a, b)
    t1.record()
    torch.cuda.synchronize()
    assert B.moe_get_status(h, dw.ws.status).code == 0
    fused = statistics.median(a.elapsed_time(b) * 1e3 for a, b in evs)
    step_us = t0.elapsed_time(t1) * 1e3 / steps
    t_flops = dw.flops / peaks["bf16_tflops"] / 1e6
    t_comb = dw.combine_bytes / peaks["hbm_gbs"] / 1e3
    t_all = all_traffic_bytes(w) / peaks["hbm_gbs"] / 1e3
    roof = max(t_flops, t_comb)
    out = {"workload": w.name, "T": w.T, "tile": f"{w.tile_m}x{w.tile_n}", "L": w.L, "steps": steps,
           "plan": {"comm_ctas": plan.comm_ctas, "P": plan.P, "co_warps": plan.co_warps},
           "step_us": step_us, "fused_kernel_us": fused, "tflops": dw.flops / fused / 1e6,
           "roofline_us": roof, "roofline_bound": "tensor" if t_flops >= t_comb else "hbm", "roofline_frac": roof / fused,
           "hbm_all_traffic_us": t_all, "frac_of_all_traffic_bound": t_all / fused,
           "bound_us": max(roof, t_all), "frac_of_bound": max(roof, t_all) / fused,
           "r_expert": dw.info["r_expert"]}
    if counts_on_device_too:
        # the same step with the routed counts left on the device (Section III-E: no copy, no host wait; the plan
        # comes from the normalised-load estimate and the kernel reads the tile count itself)
        layer2 = B.LayerCall(h, dw.x, dw.W2, dw.idx_d, dw.wt_d, dw.ws, limits=lim, counts_on_device=True)
        for _ in range(warm):
            layer2()
        torch.cuda.synchronize()
        t0.record()
        for _ in range(steps):
            layer2()
        t1.record()
        torch.cuda.synchronize()
        assert B.moe_get_status(h, dw.ws.status).code == 0
        out["step_us_counts_on_device"] = t0.elapsed_time(t1) * 1e3 / steps
        del layer2
    del dw, layer
    torch.cuda.empty_cache()
    return out


DECODE_T = (16, 64, 256, 1024)


def run_decode(h, args, device, peaks):
    """--workload dsv2lite_decode: decode-sized token counts on the DeepSeek-V2-Lite shape, tile family chosen
    by moe_select_tile.  At these sizes every expert's W2 slice is read for a handful of rows: the bound is the
    time all HBM traffic of a launch needs (W2 dominates), not the FLOPs or the combine bytes."""
    from dataclasses import replace
    from paper_2609_07536_b200 import binding as B
    from paper_2609_07536_b200 import workloads as wl
    rows = []
    for T in DECODE_T:
        w = replace(wl.DSV2L, name=f"dsv2lite_decode_T{T}", T=T)
        shape = B.make_shape(w.T, w.H, w.I, w.E_tot, w.k_tot, w.TP, w.EP, w.L)
        tm, tn = B.moe_select_tile(h, shape)
        rows.append(quick_config(h, replace(w, tile_m=tm, tile_n=tn), device, peaks, steps=max(20, args.steps), warm=max(3, args.warmup),
                                 counts_on_device_too=True))
    main = rows[2]   # T = 256
    w = replace(wl.DSV2L, name="dsv2lite_decode", T=main["T"])
    idx, wt, info = wl.make_routing(w)
    print(json.dumps({
        "metric": METRIC, "value": main["step_us"], "unit": "us/layer", "n_gpus": 1, "steps": main["steps"],
        "warmup": max(3, args.warmup), "ms_per_step": main["step_us"] / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": dict(config_of(replace(w, tile_m=int(main["tile"].split("x")[0]), tile_n=int(main["tile"].split("x")[1])), info, 1),
                       T_list=list(DECODE_T), value_is_for_T=main["T"]),
        "roofline": {"bound": "hbm", "achieved": all_traffic_bytes(w) / main["fused_kernel_us"] / 1e3, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": main["frac_of_all_traffic_bound"], "traffic": None,
                     "peak_source": peaks["source"] + ": copy bandwidth; bytes = ALL HBM traffic of a launch (x, W2, Y written "
                                    "and read back, out): at decode sizes the weights dominate, the headline roofline "
                                    "(FLOPs or combine bytes) does not bound these launches",
                     "kernel": "moe_gemm2_combine_kernel", "kernel_us": main["fused_kernel_us"]},
        "decode": rows, "cpu_baseline": None, "e2e": None,
        "gpu_launches": 2 * main["steps"],      # one routing launch (single-CTA build at these sizes) + the fused launch
    }))


# ----------------------------------------------------------------------------- per-CTA timeline
# Reader of the records the instrumented build (libmoe_b200_timeline.so) writes; slot numbers as in
# csrc/gemm2_combine.cu.

TL = dict(begin=0, role=1, first_acc=2, mma_end=3, tiles=4, wait_operand=5, issue=6, wait_tmem=7, mma_cycles=8,
          compute_end=9, cta_end=10, epi_wait=11, epi_work=12, producer_wait=13, comm_units=14, comm_wait_ns=15, co=16,
          pub_wait=32, pub_fence=33, epi_pub_wait=34, stage_late=35)


def gemm_only_mma_record(h, dw, step, occ, lim):
    """One recorded GEMM-only launch on all SMs: cycles of the MMA-issuing thread per k-block and the SM clock
    the launch ran at (those cycles over the time they took)."""
    import numpy as np
    import torch
    B, w = dw.B, dw.w
    slots = B.MOE_TIMELINE_SLOTS
    n_words = (lim.G + 2) * slots + B.MOE_MAX_L
    buf = torch.zeros(n_words, dtype=torch.int64, device=dw.x.device)
    B.moe_set_timeline(h, buf, n_words * 8)
    step(0, mode=B.MOE_MODE_GEMM_ONLY, P_override=lim.G // occ.comp_slot_sms)
    torch.cuda.synchronize()
    B.moe_set_timeline(h, None, 0)
    rec = buf.cpu().numpy().astype(np.uint64)[:lim.G * slots].reshape(lim.G, slots).astype(np.float64)
    comp = rec[rec[:, TL["tiles"]] > 0]
    if not comp.size:
        return None
    kb = comp[:, TL["tiles"]] * (-(-(w.I // w.TP) // 64))
    med = lambda v: float(np.median(v))
    return {"cycles_per_kblock": med(comp[:, TL["mma_cycles"]] / kb), "waiting_for_operands": med(comp[:, TL["wait_operand"]] / kb),
            "issuing": med(comp[:, TL["issue"]] / kb), "waiting_for_accumulator_buffer": med(comp[:, TL["wait_tmem"]] / kb),
            "sm_clock_ghz": med(comp[:, TL["mma_cycles"]] / np.maximum(1.0, comp[:, TL["mma_end"]] - comp[:, TL["begin"]])),
            "share_of_kblocks_whose_stage_was_not_ready": med(comp[:, TL["stage_late"]] / kb) if w.tile_m == 256 else None}


def run_timeline(h, dw, step, occ, lim, args):
    """One recorded fused launch (after warm-up launches): where the time of the compute CTAs goes, when the
    splits complete and what the communication warps serve while the GEMM is still running."""
    import numpy as np
    import torch
    B, w = dw.B, dw.w
    slots = B.MOE_TIMELINE_SLOTS
    n_words = (lim.G + 2) * slots + B.MOE_MAX_L
    buf = torch.zeros(n_words, dtype=torch.int64, device=dw.x.device)
    kw = dict(C_override=0, P_override=lim.G // occ.comp_slot_sms) if args.no_comm_ctas else {}
    for _ in range(max(1, args.warmup)):
        step(args.force_C, **kw)
    torch.cuda.synchronize()
    B.moe_set_timeline(h, buf, n_words * 8)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    plan, counts = step(args.force_C, ev_before=a, ev_after=b, **kw)
    torch.cuda.synchronize()
    B.moe_set_timeline(h, None, 0)
    kernel_us = a.elapsed_time(b) * 1e3
    pair = w.tile_m == 256
    grid = (((plan.comm_ctas + 1) & ~1) + 2 * plan.P) if pair else plan.comm_ctas + plan.P
    raw = buf.cpu().numpy().astype(np.uint64)
    rec = raw[:grid * slots].reshape(grid, slots).astype(np.float64)
    splits = raw[grid * slots:grid * slots + w.L].astype(np.float64)
    t0 = rec[:, TL["begin"]][rec[:, TL["begin"]] > 0].min()
    comp = rec[(rec[:, TL["role"]] == 1) & (rec[:, TL["tiles"]] > 0)]      # CTAs that issued MMAs (pair: the leaders)
    allc = rec[rec[:, TL["role"]] == 1]

    def rel(v):   # ns stamps -> us after the first CTA began
        v = v[v > 0]
        return {"min": float((v.min() - t0) / 1e3), "median": float((np.median(v) - t0) / 1e3),
                "max": float((v.max() - t0) / 1e3)} if v.size else None

    K = w.I // w.TP
    num_kb = -(-K // 64)
    kb = comp[:, TL["tiles"]] * num_kb
    per_kb = lambda slot: float(np.median(comp[:, TL[slot]] / kb)) if comp.size else None
    out = {
        "timeline": w.name, "tile": f"{w.tile_m}x{w.tile_n}", "L": w.L, "C": plan.comm_ctas, "P": plan.P,
        "co_warps": plan.co_warps, "kernel_us": kernel_us, "num_kb": num_kb,
        "cta_begin_us": rel(rec[:, TL["begin"]]), "first_accumulator_us": rel(comp[:, TL["first_acc"]]),
        "last_mma_us": rel(comp[:, TL["mma_end"]]), "compute_role_end_us": rel(allc[:, TL["compute_end"]]),
        "cta_end_us": rel(rec[:, TL["cta_end"]]),
        "split_complete_us": [float((t - t0) / 1e3) if t > 0 else None for t in splits],
        "tiles_per_cta": {"min": float(comp[:, TL["tiles"]].min()), "max": float(comp[:, TL["tiles"]].max())} if comp.size else None,
        "mma_thread_cycles_per_kblock": {"total": per_kb("mma_cycles"), "waiting_for_operands": per_kb("wait_operand"),
                                         "issuing": per_kb("issue"), "waiting_for_accumulator_buffer": per_kb("wait_tmem")},
        "epilogue_warp_cycles_per_tile": {
            "waiting": float(np.median(allc[:, TL["epi_wait"]] / np.maximum(1, comp[:, TL["tiles"]].mean()))),
            "working": float(np.median(allc[:, TL["epi_work"]] / np.maximum(1, comp[:, TL["tiles"]].mean())))} if allc.size else None,
        "publisher_cycles_per_tile": {
            "waiting_for_the_epilogue": float(np.median(allc[:, TL["pub_wait"]]) / max(1.0, float(comp[:, TL["tiles"]].mean()))),
            "fence_and_flag": float(np.median(allc[:, TL["pub_fence"]]) / max(1.0, float(comp[:, TL["tiles"]].mean()))),
            "epilogue_warp_waiting_for_the_publisher": float(np.median(allc[:, TL["epi_pub_wait"]]) / max(1.0, float(comp[:, TL["tiles"]].mean())))} if allc.size else None,
        "producer_wait_cycles_per_kblock": float(np.median(allc[:, TL["producer_wait"]]) / max(1.0, float(np.median(kb)))) if comp.size else None,
        # the SM clock the launch really ran at: cycles of the MMA thread's loop over the time it took
        "sm_clock_ghz_during_gemm": float(np.median(comp[:, TL["mma_cycles"]] / np.maximum(1.0, comp[:, TL["mma_end"]] - comp[:, TL["begin"]]))) if comp.size else None,
    }
    Q = w.k_tot * w.TP
    slab = 1024
    while slab > 8 and Q * slab * 2 > 8192:
        slab //= 2
    unit_bytes = Q * min(slab, -(-w.H // w.L)) * 2
    if plan.co_warps > 0 and allc.size:
        co = allc[:, TL["co"]:TL["co"] + 8 * plan.co_warps].reshape(-1, 8)
        units = co[:, 2]
        by_split = co[:, 4:8].sum(axis=0)
        gemm_end = np.median(comp[:, TL["mma_end"]])
        # units a warp served before the median compute CTA issued its last MMA, taking its service as even in time
        span = np.maximum(1.0, co[:, 1] - co[:, 0])
        early = np.clip((gemm_end - co[:, 0]) / span, 0.0, 1.0) * units
        out["co_resident_warps"] = {
            "warps": int(co.shape[0]), "units_total": float(units.sum()), "units_by_split": [float(v) for v in by_split[:w.L]],
            "bytes_total": float(units.sum() * unit_bytes), "units_before_median_last_mma": float(early.sum()),
            "bytes_before_median_last_mma": float(early.sum() * unit_bytes),
            "first_unit_us": rel(co[:, 0]), "last_unit_us": rel(co[:, 1]),
            "asleep_us_per_warp_median": float(np.median(co[:, 3]) / 1e3),
            "gb_per_s_per_warp_while_serving": float(np.median(units * unit_bytes / span)),
        }
    out["units_all_splits"] = w.T * w.L * (-(-(-(-w.H // w.L)) // min(slab, -(-w.H // w.L))))
    out["unit_bytes"] = unit_bytes
    print(json.dumps(out))


# ----------------------------------------------------------------------------- up-stream stage (next row)

def time_gemm1(h, dw, torch, n_warm=3, n_samples=9, cpu_rows=0):
    """Gather + grouped GEMM1 + gated activation producing x_routed (Section II-A, steps 1-2), timed alone with
    CUDA events on the workload's routing.  Not part of `value`: the paper leaves this stage unchanged."""
    from paper_2609_07536_b200 import binding as B
    from paper_2609_07536_b200 import workloads as wl
    w = dw.w
    g = torch.Generator(device=dw.x.device).manual_seed(w.data_seed + 101)
    hidden = torch.randn((w.T, w.H), generator=g, device=dw.x.device).bfloat16()
    W1 = (torch.randn((w.E_tot, 2, w.I, w.H), generator=g, device=dw.x.device) * 0.02).bfloat16()
    hr = torch.empty(B.moe_gemm1_workspace_bytes(dw.shape), dtype=torch.uint8, device=dw.x.device)
    xr = torch.empty((w.R, w.I), dtype=torch.bfloat16, device=dw.x.device)
    B.moe_build_routing(h, dw.idx_d, dw.shape, w.tile_m, dw.ws.routing, dw.ws.tile_counts, dw.ws.status)
    torch.cuda.synchronize()
    S = int(dw.ws.tile_counts[w.E_tot])
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_samples)]
    for i in range(n_warm + n_samples):
        if i >= n_warm:
            evs[i - n_warm][0].record()
        B.moe_gemm1_act(h, hidden, W1, dw.shape, w.tile_m, dw.ws.routing, S, hr, xr, dw.ws.status)
        if i >= n_warm:
            evs[i - n_warm][1].record()
    torch.cuda.synchronize()
    assert B.moe_get_status(h, dw.ws.status).code == 0
    us = statistics.median(a.elapsed_time(b) * 1e3 for a, b in evs)
    # the whole post-router layer (routing build -> GEMM1 + activation -> plan -> GEMM2 + combine), one call per step
    W2 = dw.W2
    lay = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_samples)]
    for i in range(n_warm + n_samples):
        if i >= n_warm:
            lay[i - n_warm][0].record()
        B.moe_post_router_layer(h, hidden, W1, W2, dw.idx_d, dw.wt_d, dw.ws, hr, xr)
        if i >= n_warm:
            lay[i - n_warm][1].record()
    torch.cuda.synchronize()
    assert B.moe_get_status(h, dw.ws.status).code == 0
    layer_us = statistics.median(a.elapsed_time(b) * 1e3 for a, b in lay)
    flops = 4.0 * w.R * w.H * w.I
    res = {"us": us, "tflops": flops / us / 1e6, "flops": flops,
           "bytes_gather": 2.0 * w.R * w.H * 2, "launches": 2,
           "post_router_layer_us": layer_us, "post_router_layer_launches": 7,
           "what": "gather + grouped GEMM1 (gate, up) + silu(gate) * up -> x_routed; timed alone (burst peak applies)"}
    if cpu_rows > 0:   # the oracle of this stage on a seeded sample of routed rows: parity check and CPU time
        import numpy as np
        from oracle import gemm1_act_ref as g1
        from oracle import gemm2_combine_ref as g2
        from oracle import routing_ref as rr
        rows = np.sort(np.random.default_rng(0).choice(w.R, size=min(w.R, cpu_rows), replace=False)).astype(np.int32)
        perm = rr.build_routing(dw.idx, w.E_tot, w.tile_m)["perm"]
        hb, Wb = wl.bf16_bits(hidden.cpu()), wl.bf16_bits(W1.cpu())
        t0 = time.perf_counter()
        ref = g1.gemm1_act(hb, Wb, dw.idx, perm, rows=rows)
        dt = time.perf_counter() - t0
        got = xr.float().cpu().numpy()[rows]
        rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
        tol = 1e-2 * rms + 1e-3 + 2.0 ** -8 * np.abs(ref)
        res["cpu_oracle"] = {"value": dt / len(rows) * w.R * 1e6, "unit": "us/layer", "cores": g2.threads(), "kind": "oracle",
                             "sample": f"{len(rows)} of {w.R} routed rows in {dt:.2f} s, scaled by R/n"}
        res["parity_on_sample"] = {"rows": int(len(rows)), "max_abs_err": float(np.max(np.abs(got - ref))),
                                   "within_tolerance": bool(np.all(np.abs(got - ref) <= tol))}
    return res


# ----------------------------------------------------------------------------- CPU baseline

def cpu_baseline(w, idx, wt, x_cpu, W2_cpu, budget_s=15.0):
    """The oracle's plain loops on this machine's cores over a bounded token sample, scaled
    linearly to the whole batch (cost per token is uniform: k_tot * H * I multiply-adds)."""
    import numpy as np
    from oracle import gemm2_combine_ref as ref
    from oracle import routing_ref as rr
    from paper_2609_07536_b200 import workloads as wl
    r = rr.build_routing(idx, w.E_tot, w.tile_m)
    xb, Wb = wl.bf16_bits(x_cpu), wl.bf16_bits(W2_cpu)
    cores = ref.threads()
    rng = np.random.default_rng(0)
    probe = np.sort(rng.choice(w.T, size=min(w.T, max(cores, 16)), replace=False)).astype(np.int32)
    t0 = time.perf_counter()
    ref.gemm2_combine(xb, Wb, idx, wt, r["inv_perm"], tokens=probe)
    per_tok = (time.perf_counter() - t0) / len(probe)
    n = int(max(len(probe), min(w.T, budget_s / max(per_tok, 1e-9))))
    toks = np.sort(rng.choice(w.T, size=n, replace=False)).astype(np.int32)
    t0 = time.perf_counter()
    ref.gemm2_combine(xb, Wb, idx, wt, r["inv_perm"], tokens=toks)
    dt = time.perf_counter() - t0
    us_layer = dt / n * w.T * 1e6
    # the same loops on one thread, on a small sample (about 2 s)
    n1 = int(max(4, min(n, 2.0 / max(per_tok * cores, 1e-9))))
    before = ref.set_threads(1)
    try:
        t0 = time.perf_counter()
        ref.gemm2_combine(xb, Wb, idx, wt, r["inv_perm"], tokens=toks[:n1])
        dt1 = time.perf_counter() - t0
    finally:
        ref.set_threads(before)
    return {"value": us_layer, "unit": "us/layer", "cores": cores, "kind": "oracle",
            "sample": f"{n} of {w.T} tokens (seeded random sample) timed in {dt:.2f} s, scaled by T/n; "
                      f"routing reference not included",
            "single_thread": {"value": dt1 / n1 * w.T * 1e6, "unit": "us/layer",
                              "sample": f"{n1} tokens in {dt1:.2f} s, scaled by T/n"}}, dt


def reference_arm(args):
    """--impl reference: the CPU oracle as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_07536_b200 import workloads as wl
    w = wl.CONFIGS[args.workload]
    idx, wt, info = wl.make_routing(w)
    x, W2 = wl.make_data(w)
    steps, warm = max(1, args.steps), max(0, args.warmup)
    budget = min(20.0, 150.0 / (steps + warm))
    vals = []
    base = None
    for i in range(warm + steps):
        base, dt = cpu_baseline(w, idx, wt, x, W2, budget_s=budget)
        if i >= warm:
            vals.append(base["value"])
    v = statistics.median(vals)
    base["value"] = v
    base["extrapolated"] = True
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "us/layer", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": v / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(w, info, int(os.environ.get("WORLD_SIZE", "1"))),
        "extrapolated": True,
        "note": "each of the `steps` steps times the oracle on a bounded seeded token sample and scales it by T/n "
                "(`cpu_baseline.sample` says how many tokens the last one ran); value and ms_per_step are that "
                "extrapolation to a whole layer, not the wall time of a step",
        "cpu_baseline": base,
        "e2e": {"value": v, "unit": "us/layer", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- main arm

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="dsv2lite")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-regret", action="store_true")
    ap.add_argument("--only", default="", choices=["", "fused", "gemm_only", "combine_only", "gemm1"],
                    help="time just this launch mode (for profiling): warmup + steps launches, short JSON")
    ap.add_argument("--force-C", type=int, default=0, help="with --only: communication CTAs (0 = analytical)")
    ap.add_argument("--data", default="seeded", choices=["seeded", "device"])
    ap.add_argument("--tile", default="", help="GEMM tile MxN overriding the workload's (e.g. 256x256)")
    ap.add_argument("--L", type=int, default=0, help="pipeline splits overriding the workload's")
    ap.add_argument("--T", type=int, default=0, help="token count overriding the workload's (small-T studies)")
    ap.add_argument("--calibrate", action="store_true",
                    help="one-time service-rate characterisation of the kernel family (Eq. 13): prints rho_ref")
    ap.add_argument("--sweep", action="store_true", help="selector-regret sweep on the DeepSeek-V2-Lite shape")
    ap.add_argument("--sweep-out", default="sweep.json")
    ap.add_argument("--sweep-filter", default="", help="substring a sweep workload name must contain")
    ap.add_argument("--sweep-curves", action="store_true", help="keep every t(C) in the sweep output")
    ap.add_argument("--sweep-samples", type=int, default=5, help="timed samples per C in the sweep")
    ap.add_argument("--sweep-modes", default="both", choices=["both", "static", "drain_help"])
    ap.add_argument("--counts", default="host", choices=["host", "device"],
                    help="host: tile counts copied to the host, exact plan (default); device: no copy and no wait, "
                         "plan from the normalised-load estimate (Section III-E)")
    ap.add_argument("--co-warps", type=int, default=-1,
                    help="co-resident communication warps per compute CTA (-1: the selector decides)")
    ap.add_argument("--no-comm-ctas", action="store_true",
                    help="with --only fused: launch without any dedicated communication CTA (C = 0, every SM computes)")
    ap.add_argument("--dep-model", type=int, default=0, choices=[0, 1],
                    help="static partition: 0 = readiness per split (Eq. 9 as printed), 1 = per communication tile")
    ap.add_argument("--drain-help", type=int, default=1, choices=[0, 1],
                    help="1 (default): compute CTAs help with the communication tail; 0: the paper's static partition")
    ap.add_argument("--probe", type=int, default=0,
                    help="with --timeline: time GEMM-only launches with part of the data movement left out (bits: 1 = no W2 "
                         "tile on every second k-block, 2 = no W2 tile at all, 4 = no Y stores, 8 = no x tile on pair tiles, 16 = pair tiles: MMAs issued without operand barriers, 32 = pair tiles: the MMA-issuing thread idles 200 cycles per k-block); results are garbage, only "
                         "the time means something")
    ap.add_argument("--timeline", action="store_true",
                    help="run the instrumented build (libmoe_b200_timeline.so, built on demand) and print where the "
                         "time of one fused launch goes per CTA role; honours --force-C / --no-comm-ctas / --co-warps / --L / --tile")
    args = ap.parse_args()
    if args.impl == "reference":
        return reference_arm(args)
    if args.timeline:
        from paper_2609_07536_b200 import binding as B0
        from paper_2609_07536_b200 import build as lib_build
        lib_build.build(timeline=True)
        B0.use_timeline_library()

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2609_07536_b200 import binding as B
    from paper_2609_07536_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the operator has no CPU path")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))
    h = B.moe_create(local)
    peaks = load_peaks()

    if args.sweep:
        return run_sweep(h, args, peaks)
    if args.calibrate:
        tile = tuple(int(v) for v in args.tile.split("x")) if args.tile else (128, 256)
        return calibrate(h, device, tile=tile)

    if args.workload == "dsv2lite_decode":
        run_decode(h, args, device, peaks)
        B.moe_destroy(h)
        return
    w = wl.CONFIGS[args.workload]
    if args.tile:
        from dataclasses import replace
        tm, tn = (int(v) for v in args.tile.split("x"))
        w = replace(w, tile_m=tm, tile_n=tn)
    if args.L:
        from dataclasses import replace
        w = replace(w, L=args.L)
    if args.T:
        from dataclasses import replace
        w = replace(w, T=args.T, name=f"{w.name}_T{args.T}")
    dw = DeviceWorkload(w, device, data=args.data if (args.only or args.timeline) else "seeded")
    step, (occ, lim, rho) = make_stepper(h, dw, limits_override=dict(drain_help=args.drain_help,
                                                                      force_co_warps=args.co_warps))
    K, W = max(1, args.steps), max(3, args.warmup)

    if args.timeline and args.probe:
        res = {}
        for bits in (0, args.probe):
            B.moe_set_probe(h, bits)
            ts = time_fused(step, torch, 0, 3, 9, mode=B.MOE_MODE_GEMM_ONLY, P_override=lim.G // occ.comp_slot_sms)
            res["gemm_only_us" if bits == 0 else f"gemm_only_us_probe_{bits}"] = statistics.median(ts)
            res["mma_thread" if bits == 0 else f"mma_thread_probe_{bits}"] = gemm_only_mma_record(h, dw, step, occ, lim)
        B.moe_set_probe(h, 0)
        print(json.dumps({"probe": args.probe, "workload": w.name, "tile": f"{w.tile_m}x{w.tile_n}", **res}))
        B.moe_destroy(h)
        return
    if args.timeline:
        run_timeline(h, dw, step, occ, lim, args)
        B.moe_destroy(h)
        return
    if args.only == "gemm1":
        res = time_gemm1(h, dw, torch, n_warm=max(1, args.warmup), n_samples=K)
        print(json.dumps({"only": "gemm1", "workload": w.name, **res}))
        B.moe_destroy(h)
        return
    if args.only:
        mode = {"fused": B.MOE_MODE_FUSED, "gemm_only": B.MOE_MODE_GEMM_ONLY,
                "combine_only": B.MOE_MODE_COMBINE_ONLY}[args.only]
        kw = {}
        if args.only == "gemm_only":
            kw = dict(P_override=((lim.G - args.force_C) if args.force_C else lim.G) // occ.comp_slot_sms)
        elif args.only == "combine_only":
            kw = dict(C_override=args.force_C or lim.G)
        elif args.no_comm_ctas:
            kw = dict(C_override=0, P_override=lim.G // occ.comp_slot_sms)
        if args.only == "combine_only":   # Y must exist
            step(0, mode=B.MOE_MODE_GEMM_ONLY, P_override=lim.G // occ.comp_slot_sms)
        ts = time_fused(step, torch, (args.force_C if args.only == "fused" else (1 if args.only == "combine_only" else 0)),
                        args.warmup, K, mode=mode, **kw)
        med = statistics.median(ts)
        print(json.dumps({"only": args.only, "workload": w.name, "force_C": 0 if args.no_comm_ctas else args.force_C,
                          "co_warps": args.co_warps, "L": w.L, "tile": f"{w.tile_m}x{w.tile_n}", "us": med,
                          "min_us": min(ts), "tflops": dw.flops / med / 1e6, "combine_gbs": dw.combine_bytes / med / 1e3}))
        B.moe_destroy(h)
        return

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: EXACTLY K steps between two barriers.  One step = one moe_layer call:
    # routing build -> tile counts on the host -> plan_partition -> fused launch.
    lim.force_comm_ctas = 0
    layer = B.LayerCall(h, dw.x, dw.W2, dw.idx_d, dw.wt_d, dw.ws, limits=lim, counts_on_device=(args.counts == "device"))
    for _ in range(W):
        plan = layer()
    fused_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in fused_ev:          # create the CUDA event handles
        a.record(); b.record()
    t_beg, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    wall0 = time.perf_counter()
    t_beg.record()
    for i in range(K):
        plan = layer(fused_ev[i][0], fused_ev[i][1])
    t_end.record()
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()
    step_us = t_beg.elapsed_time(t_end) * 1e3 / K
    fused_us = [a.elapsed_time(b) * 1e3 for a, b in fused_ev]
    fused_med = statistics.median(fused_us)
    # 95% interval of that median: block-stratified bootstrap (blocks of consecutive steps keep the slow
    # drift of the power-capped clock inside a block), 1000 resamples, seeded
    import random as _random
    _rng = _random.Random(0)
    _blk = max(1, len(fused_us) // 10)
    _blocks = [fused_us[i:i + _blk] for i in range(0, len(fused_us), _blk)]
    _meds = sorted(statistics.median([v for b in _blocks for v in (_rng.choice(b) for _ in b)]) for _ in range(1000))
    fused_ci = [_meds[25], _meds[974]]
    st = B.moe_get_status(h, dw.ws.status)
    assert st.code == 0
    counts = dw.ws.tile_counts[:w.E_tot + 1].tolist()

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed)
    nbytes = B.moe_host_arena_bytes(dw.shape, w.tile_m, w.tile_n)
    arena = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
    arena_ptr = arena.data_ptr() + (-arena.data_ptr()) % 256
    xh, ih, wh = dw.x_cpu.pin_memory(), torch.from_numpy(dw.idx).pin_memory(), torch.from_numpy(dw.wt).pin_memory()
    counts_pin = torch.zeros(w.E_tot + 1, dtype=torch.int32).pin_memory()
    out_h = torch.empty((w.T, w.H), dtype=torch.bfloat16).pin_memory()
    Ke = max(3, min(K, 20))
    for _ in range(3):
        B.moe_layer_host(h, xh, ih, wh, dw.W2, dw.shape, w.tile_m, w.tile_n, None, arena_ptr, nbytes, counts_pin, out_h)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(Ke):
        B.moe_layer_host(h, xh, ih, wh, dw.W2, dw.shape, w.tile_m, w.tile_n, None, arena_ptr, nbytes, counts_pin, out_h)
    ev1.record()
    barrier()
    e2e_us = ev0.elapsed_time(ev1) * 1e3 / Ke     # device time from the first copy to the last read-back
    del arena
    h2d = xh.numel() * 2 + ih.numel() * 4 + wh.numel() * 4
    d2h = out_h.numel() * 2 + (w.E_tot + 1) * 4 + 16

    # ---- max over ranks
    step_us, fused_med, e2e_us = max_over_ranks([step_us, fused_med, e2e_us], world, device)

    extra = {}
    if rank == 0:
        # ---- the two roles alone (all SMs compute / all SMs communicate)
        G_sm = lim.G
        gemm_only = statistics.median(time_fused(step, torch, 0, 2, 7, mode=B.MOE_MODE_GEMM_ONLY,
                                                 P_override=G_sm // occ.comp_slot_sms))
        lim_all = G_sm
        comb_only = statistics.median(time_fused(step, torch, 1, 2, 7, mode=B.MOE_MODE_COMBINE_ONLY, C_override=G_sm))
        extra["gemm_only"] = {"us": gemm_only, "tflops": dw.flops / gemm_only / 1e6,
                              "frac_of_bf16_peak": dw.flops / gemm_only / 1e6 / peaks["bf16_tflops"], "P": G_sm}
        extra["combine_only"] = {"us": comb_only, "gbs": dw.combine_bytes / comb_only / 1e3,
                                 "frac_of_hbm_peak": dw.combine_bytes / comb_only / 1e3 / peaks["hbm_gbs"], "C": lim_all}
        # ---- selector regret on this workload: every feasible C timed
        if not args.no_regret:
            extra["regret"] = regret_of_workload(step, torch, counts, lim, (plan.comm_ctas, plan.co_warps), n_warm=1, n_samples=5)
            # the paper's static partition on the same workload: its pick, its sweep, its regret
            step0, (occ0, lim0, rho0) = make_stepper(h, dw, limits_override=dict(drain_help=1 - args.drain_help))
            lim0.force_comm_ctas = 0
            plan0 = B.plan_partition(counts[:w.E_tot], occ0, lim0, dw.shape, rho0)
            key = "regret_static_partition" if args.drain_help else "regret_drain_help"
            extra[key] = regret_of_workload(step0, torch, counts, lim0, (plan0.comm_ctas, plan0.co_warps), n_warm=1, n_samples=5)
        # ---- solver overhead: mean over >= 1e6 calls, rotating routed-count vectors
        rng = np.random.default_rng(0)
        base_counts = np.array(counts[:w.E_tot])
        sets = [np.maximum(0, base_counts + rng.integers(-3, 4, size=w.E_tot)).tolist() for _ in range(64)]
        lim.force_comm_ctas = 0
        extra["solver_ns"] = B.moe_time_plan_partition(sets, occ, lim, dw.shape, rho, 1_000_000)
        if not args.no_cpu_baseline:
            extra["cpu_baseline"], _ = cpu_baseline(w, dw.idx, dw.wt, dw.x_cpu, dw.W2_cpu)
        # ---- context: the library GEMM (cuBLAS through torch.matmul) on a dense problem with the same FLOPs and the
        # same contraction length K = I / TP: [R * TP, K] x [K, H].  Not part of the operator: it says what a dense
        # GEMM without routing, padding, scattered stores and flags reaches at this K on this GPU.
        a_ = torch.randn((w.R * w.TP, w.I // w.TP), device=device, dtype=torch.bfloat16)
        b_ = torch.randn((w.H, w.I // w.TP), device=device, dtype=torch.bfloat16)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(9)]
        for _ in range(2):
            c_ = a_ @ b_.t()
        for ea, eb in evs:
            ea.record(); c_ = a_ @ b_.t(); eb.record()
        torch.cuda.synchronize()
        cub = statistics.median(ea.elapsed_time(eb) * 1e3 for ea, eb in evs)
        extra["context_cublas_same_flops"] = {
            "shape": [w.R * w.TP, w.H, w.I // w.TP], "us": cub, "tflops": dw.flops / cub / 1e6,
            "gemm_only_over_cublas": cub / extra["gemm_only"]["us"],
            "what": "torch.matmul (cuBLAS) on a dense bf16 GEMM of the same FLOPs and K, timed alone; context, not a target"}
        del a_, b_, c_
        torch.cuda.empty_cache()
        # ---- the other named workloads, briefly (a second or two each): fused time and roofline fractions
        if args.workload == "dsv2lite" and not args.tile and not args.T and not args.L:
            # the other two shapes of the task, each with the tile family the library's dispatch picks for it
            from dataclasses import replace as _replace
            others = []
            for n in ("granite3moe", "qwen15moe"):
                wo = wl.CONFIGS[n]
                tm, tn = B.moe_select_tile(h, B.make_shape(wo.T, wo.H, wo.I, wo.E_tot, wo.k_tot, wo.TP, wo.EP, wo.L))
                others.append(quick_config(h, _replace(wo, tile_m=tm, tile_n=tn), device, peaks))
            extra["other_configs"] = others
        # ---- the up-stream stage (next row of the scope table), reported beside the headline, not in it
        g1res = time_gemm1(h, dw, torch, cpu_rows=0 if args.no_cpu_baseline else 4096)
        g1res["frac_of_bf16_peak"] = g1res["tflops"] / peaks["bf16_tflops"]
        extra["gemm1_act"] = g1res

    if rank == 0:
        tf_peak, tf_rule = tensor_peak_for(peaks, K * step_us / 1e6, clocks)
        t_flops_us = dw.flops / tf_peak / 1e6
        t_hbm_us = dw.combine_bytes / peaks["hbm_gbs"] / 1e3
        tensor_bound = t_flops_us >= t_hbm_us
        ach = dw.flops / fused_med / 1e6 if tensor_bound else dw.combine_bytes / fused_med / 1e3
        peak = tf_peak if tensor_bound else peaks["hbm_gbs"]
        tf_sust = peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"]
        roofline = {
            "bound": "tensor" if tensor_bound else "hbm", "achieved": ach, "peak": peak,
            "unit": "TFLOP/s" if tensor_bound else "GB/s", "frac": ach / peak, "traffic": None,
            "peak_source": peaks["source"] + (": " + tf_rule if tensor_bound else ": copy bandwidth"),
            "kernel": "moe_gemm2_combine_pair_kernel" if w.tile_m == 256 else "moe_gemm2_combine_kernel",
            "kernel_us": fused_med, "kernel_us_ci95": fused_ci, "roofline_us": max(t_flops_us, t_hbm_us),
            "frac_of_burst_peak": (ach / peaks["bf16_tflops"]) if tensor_bound else None,
            "burst_peak": peaks["bf16_tflops"] if tensor_bound else None,
            "frac_of_sustained_peak": (ach / tf_sust) if tensor_bound else None,
            "sustained_peak": tf_sust if tensor_bound else None,
        }
        # DRAM read + write bytes of one fused launch from the ncu capture summarised in
        # profiles/fused_gemm2_combine_dsv2lite_ncu.md (same workload, same launch configuration)
        x_passes = 1 if (args.drain_help and plan.co_warps == 0) else w.L   # m-tile-major order reads x once, split-major once per split
        all_bytes = all_traffic_bytes(w, x_passes)
        # every byte the launch has to move through HBM (x, W2, Y written and read back, out): not part of the
        # headline roofline, but the real bound at small T, where every expert's weights are read for a few rows
        roofline["hbm_all_traffic_us"] = all_bytes / peaks["hbm_gbs"] / 1e3
        if w.name in NCU_TRAFFIC_BYTES and (w.tile_m, w.tile_n, w.L, plan.co_warps) == NCU_TRAFFIC_BYTES[w.name][1]:
            roofline["traffic"] = NCU_TRAFFIC_BYTES[w.name][0]
            roofline["traffic_algorithmic"] = all_bytes
        line = {
            "metric": METRIC, "value": job_value(step_us, world), "unit": "us/layer", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": step_us / 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(w, dw.info, world),
            "plan": {"comm_ctas": plan.comm_ctas, "R": plan.R, "P": plan.P, "W_comp": plan.W_comp,
                     "W_comm": plan.W_comm, "rho": plan.rho_q / 2 ** 20, "drain_help": plan.drain_help,
                     "co_warps": plan.co_warps},
            "fused_kernel_us": fused_med, "tflops": dw.flops / fused_med / 1e6,
            "wall_ms_per_step": wall * 1e3 / K,
            "roofline": roofline,
            "e2e": {"value": job_value(e2e_us, world), "unit": "us/layer", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": Ke},
            "gpu_launches": (routing_launches(w.T * w.k) + 1) * K,
            "clocks": clocks,
            "paper_context": {"hardware": "4xA100-SXM4-40GB", "mean_regret": 0.0322, "solver_us": 0.157,
                              "geomean_speedup_over_comet": 2.528},
        }
        line.update(extra)
        if "cpu_baseline" not in line:
            line["cpu_baseline"] = None
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    B.moe_destroy(h)


if __name__ == "__main__":
    main()
