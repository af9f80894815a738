#!/usr/bin/env python
"""Benchmark of the MoE expert-FFN layer (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

A step is one pass of the whole hot path (route-permute, gate/up GEMM + SwiGLU, down GEMM,
unpermute-combine, and the four backward calls) over one batch of seeded synthetic input.  The
headline workload is the largest of the five configurations ("imbalanced"); it is timed for at
least one second (the number of timed steps is raised above --steps when needed, and the line says
how many were timed).  The metric is whole-layer throughput in TFLOP/s on the algorithmic work
18*R*H*I; the JSON line also carries the grouped-GEMM-only throughput, the permute bandwidth, a
roofline object for the dominant kernel, an end-to-end number through the host-buffer entry point,
the same step run back to back for two seconds, and the fp64 oracle timed on the host cores -- all
on that workload.  The other workloads follow in `other_configs`, each timed for at least half a
second with its own roofline object.  With N > 1 (torchrun) every rank runs an independent replica of the
same workload: the layer is single-GPU by design, there is no collective on the data path.
`--impl reference` times the CPU oracle alone on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2606_26453_b200 import workloads as W

METRIC = "moe_layer_fwd_bwd_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# Tensor-pipe rate of one SM per clock (a 128x256x16 bf16 tcgen05.mma retires in 128 cycles: measured with a bare
# issue loop), used for the clock-normalised fractions.
PIPE_FLOP_PER_CLK_PER_SM = 8192.0
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of a workload's dominant grouped-GEMM
# kernel, from one ncu capture on a SCALED copy of the workload (tokens and experts divided by `scale`, same H, I,
# top-k, routing law and rows per expert), multiplied by `scale`: every operand and result of these kernels grows in
# proportion.  (workload, call) -> (bytes per full launch, which capture it comes from); absent -> null.
NCU_TRAFFIC = {
    ("imbalanced", "gateup_swiglu"): (9193.2e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("imbalanced", "down"): (3608.0e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("imbalanced", "down_dgrad"): (4548.4e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("imbalanced", "down_wgrad"): (4209.6e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("imbalanced", "gateup_dgrad"): (6412.4e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("imbalanced", "gateup_wgrad"): (8502.4e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("few_large", "gateup_swiglu"): (3594.8e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("few_large", "down"): (2325.6e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("few_large", "down_dgrad"): (1500.0e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("few_large", "down_wgrad"): (1607.2e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("few_large", "gateup_dgrad"): (4612.4e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("few_large", "gateup_wgrad"): (2831.6e6, "ncu on a 1/4 copy (tokens and experts divided by 4), scaled x 4"),
    ("fine_grained", "gateup_swiglu"): (1029.0e6, "ncu capture of the full-size workload"),
    ("fine_grained", "down"): (525.0e6, "ncu capture of the full-size workload"),
    ("fine_grained", "down_wgrad"): (497.6e6, "ncu capture of the full-size workload"),
    ("fine_grained", "gateup_dgrad"): (982.3e6, "ncu capture of the full-size workload"),
    ("fine_grained", "gateup_wgrad"): (939.5e6, "ncu capture of the full-size workload"),
    ("many_small", "gateup_swiglu"): (1953.2e6, "ncu capture of the full-size workload"),
    ("many_small", "down"): (1110.1e6, "ncu capture of the full-size workload"),
    ("many_small", "down_wgrad"): (1152.4e6, "ncu capture of the full-size workload"),
    ("many_small", "gateup_dgrad"): (1727.9e6, "ncu capture of the full-size workload"),
    ("many_small", "gateup_wgrad"): (1883.8e6, "ncu capture of the full-size workload"),
    ("paper_dw1", "gateup_swiglu"): (5112.0e6, "ncu on a 1/8 copy (tokens and experts divided by 8), scaled x 8"),
    ("paper_dw1", "down"): (2520.8e6, "ncu on a 1/8 copy (tokens and experts divided by 8), scaled x 8"),
    ("paper_dw1", "down_dgrad"): (2548.8e6, "ncu on a 1/8 copy (tokens and experts divided by 8), scaled x 8"),
    ("paper_dw1", "down_wgrad"): (2372.8e6, "ncu on a 1/8 copy (tokens and experts divided by 8), scaled x 8"),
    ("paper_dw1", "gateup_dgrad"): (5536.8e6, "ncu on a 1/8 copy (tokens and experts divided by 8), scaled x 8"),
    ("paper_dw1", "gateup_wgrad"): (4871.2e6, "ncu on a 1/8 copy (tokens and experts divided by 8), scaled x 8"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------------------------
# clock sampling during the timed region (read-only NVML queries)
# --------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, device_index: int, period_s: float = 0.005):
        self.samples, self.reasons, self.power = [], set(), []
        self.period = period_s
        self.stop_flag = threading.Event()
        self.thread = None
        self.max_mhz = None
        self.handle = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(device_index).uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.handle = None

    def _run(self):
        nv = self.nv
        while not self.stop_flag.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.handle) / 1000.0)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.handle is not None:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()

    def stop(self):
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None}


# --------------------------------------------------------------------------------------------
# one step of the CUDA path, as the fine-grained C-ABI calls (so every kernel can be timed)
# --------------------------------------------------------------------------------------------
CALLS = ["permute", "gateup_swiglu", "down", "combine", "combine_bwd", "down_dgrad", "down_wgrad", "swiglu_bwd",
         "gateup_dgrad", "gateup_wgrad", "permute_bwd"]
LAUNCHES_PER_CALL = {"permute": 3}
GEMM_CALLS = ["gateup_swiglu", "down", "down_dgrad", "down_wgrad", "gateup_dgrad", "gateup_wgrad"]


def call_flops(cfg):
    rhi = float(cfg.R) * cfg.H * cfg.I
    return {"gateup_swiglu": 4 * rhi, "down": 2 * rhi, "down_dgrad": 2 * rhi, "down_wgrad": 2 * rhi,
            "gateup_dgrad": 4 * rhi, "gateup_wgrad": 4 * rhi}


def call_bytes(cfg):
    T, H, I, E, K, R = cfg.T, cfg.H, cfg.I, cfg.E, cfg.K, cfg.R
    return {"permute": T * H * 2 + R * H * 2 + R * 4 + 2 * R * 4 + (2 * E + 1) * 4,
            "combine": R * H * 2 + T * H * 2 + 2 * R * 4,
            "combine_bwd": T * H * 2 + 2 * R * H * 2 + 2 * R * 4 + R * 4,
            "swiglu_bwd": R * I * 2 * 5,
            "permute_bwd": R * H * 2 + T * H * 2 + R * 4}


CALLS_FUSED = ["permute", "gateup_swiglu", "down", "combine", "combine_bwd", "down_dgrad_swiglu_bwd", "down_wgrad",
               "gateup_dgrad", "gateup_wgrad", "permute_bwd"]


def make_step(B, b, wl, fused=False):
    """One layer step as a list of C-ABI calls: CALLS, or CALLS_FUSED (the down dgrad and the SwiGLU backward as the
    one fused call)."""
    x, idx, w, dy = wl["X"], wl["topk_idx"], wl["topk_w"], wl["dY"]
    wg, wu, wd = wl["W_gate"], wl["W_up"], wl["W_down"]
    d = b.d
    table = {
        "permute": lambda: B.moe_permute(d, x, idx, b.x_perm, b.counts, b.offsets, b.row_to_pair, b.pair_to_row, b.workspace),
        "gateup_swiglu": lambda: B.moe_grouped_gemm_gateup_swiglu(d, b.x_perm, wg, wu, b.offsets, b.h_act, b.gu),
        "down": lambda: B.moe_grouped_gemm_down(d, b.h_act, wd, b.offsets, b.y_perm),
        "combine": lambda: B.moe_unpermute_combine(d, b.y_perm, w, b.pair_to_row, b.y),
        "combine_bwd": lambda: B.moe_unpermute_combine_bwd(d, dy, b.y_perm, w, b.pair_to_row, b.dy_perm, b.dtopk_w),
        "down_dgrad": lambda: B.moe_grouped_gemm_down_dgrad(d, b.dy_perm, wd, b.offsets, b.dh_act),
        "down_wgrad": lambda: B.moe_grouped_gemm_down_wgrad(d, b.h_act, b.dy_perm, b.offsets, b.dw_down),
        "swiglu_bwd": lambda: B.moe_swiglu_bwd(d, b.dh_act, b.gu, b.dgu),
        "down_dgrad_swiglu_bwd": lambda: B.moe_grouped_gemm_down_dgrad_swiglu_bwd(d, b.dy_perm, wd, b.gu, b.offsets, b.dgu),
        "gateup_dgrad": lambda: B.moe_grouped_gemm_gateup_dgrad(d, b.dgu, wg, wu, b.offsets, b.dx_perm),
        "gateup_wgrad": lambda: B.moe_grouped_gemm_gateup_wgrad(d, b.x_perm, b.dgu, b.offsets, b.dw_gate, b.dw_up),
        "permute_bwd": lambda: B.moe_permute_bwd(d, b.dx_perm, b.pair_to_row, b.dx),
    }
    fns = [table[c] for c in (CALLS_FUSED if fused else CALLS)]

    def step(events=None):
        if events is None:
            for f in fns:
                f()
            return
        events[0].record()
        for i, f in enumerate(fns):
            f()
            events[i + 1].record()

    return step


def time_fp8_step(B, cfg, res, device, min_seconds=0.5):
    """The layer step with the four row-ragged GEMMs replaced by their block-scaled FP8 twins (weight gradients, data
    movement and SwiGLU backward unchanged): permute, quantise X_perm, FP8 gate/up, SwiGLU (+ FP8 form of H_act), FP8
    down, combine | combine backward, quantise dY_perm, FP8 down dgrad, down wgrad, SwiGLU backward (+ FP8 form of dGU),
    FP8 gate/up dgrad, gate/up wgrad, permute backward.  Timed back to back for at least `min_seconds`, once with the four
    weight quantisations inside every step (weights change every optimizer step) and once with them outside (several
    micro-batches per optimizer step)."""
    if cfg.H % 128 or cfg.I % 128:
        return None
    b, wl = res["buffers"], res["wl"]
    d = b.d
    R, E, H, I = cfg.R, cfg.E, cfg.H, cfg.I
    x, idx, w, dy = wl["X"], wl["topk_idx"], wl["topk_w"], wl["dY"]
    wg, wu, wd = wl["W_gate"], wl["W_up"], wl["W_down"]
    u8 = lambda n: torch.empty(n, dtype=torch.uint8, device=device)
    xc, xs = u8(R * H), u8(B.moe_mxfp8_x_scale_bytes(d))            # also reused for dY_perm (same shape)
    hc, hs = u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    gc, gs = u8(R * 2 * I), u8(B.moe_mxfp8_dgu_scale_bytes(d))
    w_gu, s_gu = u8(E * 2 * I * H), u8(B.moe_mxfp8_w_gateup_scale_bytes(d))
    w_dn, s_dn = u8(E * H * I), u8(B.moe_mxfp8_w_down_scale_bytes(d))
    w_dd, s_dd = u8(E * I * H), u8(B.moe_mxfp8_w_down_dgrad_scale_bytes(d))
    w_gd, s_gd = u8(E * H * 2 * I), u8(B.moe_mxfp8_w_gateup_dgrad_scale_bytes(d))

    def quantise_weights():
        B.moe_mxfp8_quantize_w_gateup(d, wg, wu, w_gu, s_gu)
        B.moe_mxfp8_quantize_w_down(d, wd, w_dn, s_dn)
        B.moe_mxfp8_quantize_w_down_dgrad(d, wd, w_dd, s_dd)
        B.moe_mxfp8_quantize_w_gateup_dgrad(d, wg, wu, w_gd, s_gd)

    def step():
        B.moe_permute(d, x, idx, b.x_perm, b.counts, b.offsets, b.row_to_pair, b.pair_to_row, b.workspace)
        B.moe_mxfp8_quantize_x_perm(d, b.x_perm, xc, xs)
        B.moe_grouped_gemm_gateup_mxfp8(d, xc, xs, w_gu, s_gu, b.offsets, b.gu)
        B.moe_swiglu_mxfp8(d, b.gu, b.h_act, hc, hs)
        B.moe_grouped_gemm_down_mxfp8(d, hc, hs, w_dn, s_dn, b.offsets, b.y_perm)
        B.moe_unpermute_combine(d, b.y_perm, w, b.pair_to_row, b.y)
        B.moe_unpermute_combine_bwd(d, dy, b.y_perm, w, b.pair_to_row, b.dy_perm, b.dtopk_w)
        B.moe_mxfp8_quantize_dy_perm(d, b.dy_perm, xc, xs)
        B.moe_grouped_gemm_down_dgrad_mxfp8(d, xc, xs, w_dd, s_dd, b.offsets, b.dh_act)
        B.moe_grouped_gemm_down_wgrad(d, b.h_act, b.dy_perm, b.offsets, b.dw_down)
        B.moe_swiglu_bwd_mxfp8(d, b.dh_act, b.gu, b.dgu, gc, gs)
        B.moe_grouped_gemm_gateup_dgrad_mxfp8(d, gc, gs, w_gd, s_gd, b.offsets, b.dx_perm)
        B.moe_grouped_gemm_gateup_wgrad(d, b.x_perm, b.dgu, b.offsets, b.dw_gate, b.dw_up)
        B.moe_permute_bwd(d, b.dx_perm, b.pair_to_row, b.dx)

    def timed(fn):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        n = max(3, int(math.ceil(min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3))))
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    quantise_weights()
    ms_out = timed(step)
    y_fp8, dx_fp8 = b.y.clone(), b.dx.clone()

    def step_with_weights():
        quantise_weights()
        step()

    ms_in = timed(step_with_weights)
    # leave the buffers as the bf16 step leaves them, and measure the distance of the FP8 step's results from them
    make_step(B, b, wl)()
    torch.cuda.synchronize()
    if B.moe_device_status() != 0:
        raise RuntimeError("device status word is set after the FP8 step")
    rel = lambda a, r: float((a.float() - r.float()).norm() / r.float().norm())
    return {"layer_tflops_weights_quantised_outside": cfg.flops_fwd_bwd / (ms_out * 1e-3) / 1e12,
            "ms_per_step_weights_quantised_outside": ms_out, "ms_per_step_weights_quantised_every_step": ms_in,
            "bf16_ms_per_step": res["total_ms"] / res["steps"], "gpu_launches_per_step": 15,
            "rel_frobenius_to_bf16_step": {"Y": rel(y_fp8, b.y), "dX": rel(dx_fp8, b.dx)},
            "note": "14 library calls (permute is two launches); two activation quantisers and the forward SwiGLU are separate "
                    "HBM-bound launches here, the quantiser of dGU rides in the SwiGLU backward"}


def time_mxfp8(B, cfg, res, device, reps=20, min_seconds=0.3, warm=3):
    """The block-scaled FP8 twins of the six grouped GEMMs -- down forward, down dgrad, gate/up dgrad, gate/up forward
    (with its activation call), and the two weight gradients (both operands are activations there: `quantize_act_ms`
    covers both, `quantize_w_ms` is empty) -- on this workload's own activations, weights and offsets: per GEMM the activation quantiser, the weight quantiser (once per optimizer step in training) and the GEMM,
    each timed alone (back to back for at least `min_seconds`, events), beside the bf16 call timed the same way."""
    if cfg.H % 128 or cfg.I % 128:
        return None
    b, wl = res["buffers"], res["wl"]
    d = b.d
    R, E, H, I = cfg.R, cfg.E, cfg.H, cfg.I
    u8 = lambda n: torch.empty(n, dtype=torch.uint8, device=device)

    def timed(fn):
        for _ in range(warm):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = reps
        if min_seconds > 0:   # (profiling runs pass 0: every call is then launched exactly `warm + reps` times)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            n = max(reps, int(math.ceil(min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3))))
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    def leg(flops, bf16_fn, q_act, q_w, fp8_fn, got, want):
        o = {"bf16_ms": timed(bf16_fn), "quantize_act_ms": timed(q_act), "quantize_w_ms": timed(q_w), "fp8_ms": timed(fp8_fn)}
        o["bf16_tflops"] = flops / (o["bf16_ms"] * 1e-3) / 1e12
        o["fp8_tflops"] = flops / (o["fp8_ms"] * 1e-3) / 1e12
        o["rel_frobenius_to_bf16_result"] = float((got.float() - want.float()).norm() / want.float().norm())
        return o

    out = {}
    hc, hs = u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    wc, ws = u8(E * H * I), u8(B.moe_mxfp8_w_down_scale_bytes(d))
    yq = torch.empty_like(b.y_perm)
    out["down"] = leg(2.0 * R * H * I,
                      lambda: B.moe_grouped_gemm_down(d, b.h_act, wl["W_down"], b.offsets, b.y_perm),
                      lambda: B.moe_mxfp8_quantize_h_act(d, b.h_act, hc, hs),
                      lambda: B.moe_mxfp8_quantize_w_down(d, wl["W_down"], wc, ws),
                      lambda: B.moe_grouped_gemm_down_mxfp8(d, hc, hs, wc, ws, b.offsets, yq), yq, b.y_perm)
    del hc, hs, wc, ws, yq
    dc, ds = u8(R * H), u8(B.moe_mxfp8_dy_scale_bytes(d))
    vc, vs = u8(E * I * H), u8(B.moe_mxfp8_w_down_dgrad_scale_bytes(d))
    dhq, dh_ref = torch.empty_like(b.dh_act), torch.empty_like(b.dh_act)
    out["down_dgrad"] = leg(2.0 * R * H * I,
                            lambda: B.moe_grouped_gemm_down_dgrad(d, b.dy_perm, wl["W_down"], b.offsets, dh_ref),
                            lambda: B.moe_mxfp8_quantize_dy_perm(d, b.dy_perm, dc, ds),
                            lambda: B.moe_mxfp8_quantize_w_down_dgrad(d, wl["W_down"], vc, vs),
                            lambda: B.moe_grouped_gemm_down_dgrad_mxfp8(d, dc, ds, vc, vs, b.offsets, dhq), dhq, dh_ref)
    del dc, ds, vc, vs, dhq, dh_ref
    gc, gs = u8(R * 2 * I), u8(B.moe_mxfp8_dgu_scale_bytes(d))
    uc, us = u8(E * H * 2 * I), u8(B.moe_mxfp8_w_gateup_dgrad_scale_bytes(d))
    dxq, dx_ref = torch.empty_like(b.dx_perm), torch.empty_like(b.dx_perm)
    out["gateup_dgrad"] = leg(4.0 * R * H * I,
                              lambda: B.moe_grouped_gemm_gateup_dgrad(d, b.dgu, wl["W_gate"], wl["W_up"], b.offsets, dx_ref),
                              lambda: B.moe_mxfp8_quantize_dgu(d, b.dgu, gc, gs),
                              lambda: B.moe_mxfp8_quantize_w_gateup_dgrad(d, wl["W_gate"], wl["W_up"], uc, us),
                              lambda: B.moe_grouped_gemm_gateup_dgrad_mxfp8(d, gc, gs, uc, us, b.offsets, dxq), dxq, dx_ref)
    del gc, gs, uc, us, dxq, dx_ref
    xc, xs = u8(R * H), u8(B.moe_mxfp8_x_scale_bytes(d))
    tc, ts = u8(E * 2 * I * H), u8(B.moe_mxfp8_w_gateup_scale_bytes(d))
    hc, hs = u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    guq, hq, h_ref, gu_ref = torch.empty_like(b.gu), torch.empty_like(b.h_act), torch.empty_like(b.h_act), torch.empty_like(b.gu)

    def gateup_fp8():   # the GEMM and the activation (which also emits the FP8 form the down projection reads)
        B.moe_grouped_gemm_gateup_mxfp8(d, xc, xs, tc, ts, b.offsets, guq)
        B.moe_swiglu_mxfp8(d, guq, hq, hc, hs)

    out["gateup_swiglu"] = leg(4.0 * R * H * I,
                               lambda: B.moe_grouped_gemm_gateup_swiglu(d, b.x_perm, wl["W_gate"], wl["W_up"], b.offsets, h_ref, gu_ref),
                               lambda: B.moe_mxfp8_quantize_x_perm(d, b.x_perm, xc, xs),
                               lambda: B.moe_mxfp8_quantize_w_gateup(d, wl["W_gate"], wl["W_up"], tc, ts),
                               gateup_fp8, hq, h_ref)
    out["gateup_swiglu"]["fp8_gemm_ms"] = timed(lambda: B.moe_grouped_gemm_gateup_mxfp8(d, xc, xs, tc, ts, b.offsets, guq))
    out["gateup_swiglu"]["swiglu_and_quantize_ms"] = timed(lambda: B.moe_swiglu_mxfp8(d, guq, hq, hc, hs))
    del xc, xs, tc, ts, hc, hs, guq, hq, h_ref, gu_ref
    # the two weight gradients: operands quantised along the token axis (both are activations: no per-optimizer-step part)
    tok = lambda n: (u8(B.moe_mxfp8_tokens_codes_bytes(d, n)), u8(B.moe_mxfp8_tokens_scale_bytes(d, n)))
    (ac, asc), (bc, bsc) = tok(I), tok(H)
    dwq, dw_ref = torch.empty_like(b.dw_down), torch.empty_like(b.dw_down)

    def q_down_wgrad():
        B.moe_mxfp8_quantize_tokens(d, b.h_act, I, 0, I, b.offsets, ac, asc)
        B.moe_mxfp8_quantize_tokens(d, b.dy_perm, H, 0, H, b.offsets, bc, bsc)

    out["down_wgrad"] = leg(2.0 * R * H * I,
                            lambda: B.moe_grouped_gemm_down_wgrad(d, b.h_act, b.dy_perm, b.offsets, dw_ref),
                            q_down_wgrad, lambda: None,
                            lambda: B.moe_grouped_gemm_down_wgrad_mxfp8(d, ac, asc, bc, bsc, dwq), dwq, dw_ref)
    del ac, asc, bc, bsc, dwq, dw_ref
    (xc, xs), (gc, gs), (uc, us) = tok(H), tok(I), tok(I)
    dgq, duq = torch.empty_like(b.dw_gate), torch.empty_like(b.dw_up)
    dg_ref, du_ref = torch.empty_like(b.dw_gate), torch.empty_like(b.dw_up)

    def q_gateup_wgrad():
        B.moe_mxfp8_quantize_tokens(d, b.x_perm, H, 0, H, b.offsets, xc, xs)
        B.moe_mxfp8_quantize_tokens(d, b.dgu, 2 * I, 0, I, b.offsets, gc, gs)
        B.moe_mxfp8_quantize_tokens(d, b.dgu, 2 * I, I, I, b.offsets, uc, us)

    out["gateup_wgrad"] = leg(4.0 * R * H * I,
                              lambda: B.moe_grouped_gemm_gateup_wgrad(d, b.x_perm, b.dgu, b.offsets, dg_ref, du_ref),
                              q_gateup_wgrad, lambda: None,
                              lambda: B.moe_grouped_gemm_gateup_wgrad_mxfp8(d, xc, xs, gc, gs, uc, us, dgq, duq), dgq, dg_ref)
    del xc, xs, gc, gs, uc, us, dgq, duq, dg_ref, du_ref
    out["note"] = ("E4M3 elements, E8M0 scale per 32 along the contraction; tcgen05.mma kind::mxf8f6f4.block_scale on "
                   "256 x 208 CTA-pair tiles from 256 rows per expert on average, 128 x 128 single-CTA tiles below; "
                   "the bf16 twins run 256 x 256 CTA-pair tiles; the FP8 gate/up time is the GEMM plus the activation call, "
                   "which also writes the FP8 form of H_act (so the down projection's quantize_act_ms is not paid in a chain)")
    if B.moe_device_status() != 0:
        raise RuntimeError("device status word is set after the MXFP8 calls")
    return out


def time_fused_variant(B, cfg, res, device, seconds=0.8, rounds=4):
    """The step with moe_grouped_gemm_down_dgrad_swiglu_bwd in place of moe_grouped_gemm_down_dgrad + moe_swiglu_bwd,
    timed beside the two-call step: blocks of steps of the two forms alternate (so that both see the same power and
    clock state), events around every call."""
    b, wl = res["buffers"], res["wl"]
    forms = {"two_call": (make_step(B, b, wl), CALLS), "fused": (make_step(B, b, wl, fused=True), CALLS_FUSED)}
    ms_est = res["total_ms"] / res["steps"]
    n = max(2, int(seconds * 1e3 / ms_est / (2 * rounds)))
    tot = {k: 0.0 for k in forms}
    per = {k: {c: 0.0 for c in names} for k, (_, names) in forms.items()}
    for _ in range(2):
        forms["fused"][0]()
    for _ in range(rounds):
        for k, (step, names) in forms.items():
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)] for _ in range(n)]
            for s in range(n):
                step(evs[s])
            torch.cuda.synchronize()
            tot[k] += evs[0][0].elapsed_time(evs[-1][-1])
            for i, c in enumerate(names):
                per[k][c] += sum(e[i].elapsed_time(e[i + 1]) for e in evs)
    steps = n * rounds
    if B.moe_device_status() != 0:
        raise RuntimeError("device status word is set after the fused-variant steps")
    two, fus = tot["two_call"] / steps, tot["fused"] / steps
    return {"steps_each": steps, "two_call_ms_per_step": two, "fused_ms_per_step": fus, "step_time_ratio": fus / two,
            "fused_layer_tflops": cfg.flops_fwd_bwd / (fus * 1e-3) / 1e12,
            "down_dgrad_ms": per["two_call"]["down_dgrad"] / steps, "swiglu_bwd_ms": per["two_call"]["swiglu_bwd"] / steps,
            "down_dgrad_swiglu_bwd_ms": per["fused"]["down_dgrad_swiglu_bwd"] / steps,
            "note": "alternating blocks of the two step forms; the fused call writes dGU straight from the fp32 "
                    "accumulator (dH_act is never materialised)"}


def time_config(B, cfg, device, steps, warmup, dist=None, sample_clocks=True, min_seconds=0.0, fused=False):
    """Warm-up, then `steps` timed steps between two events (CUDA events around every call inside).  With
    min_seconds > 0 the step count is raised until the timed region lasts at least that long (estimated from three
    untimed steps after the warm-up; the maximum over ranks, so that every rank times the same count)."""
    wl = W.make_workload_device(cfg, device)
    b = B.alloc_layer_buffers(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K, device=device)
    step = make_step(B, b, wl, fused=fused)
    calls = CALLS_FUSED if fused else CALLS
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    if B.moe_device_status() != 0:
        raise RuntimeError("device status word is set after warm-up")
    if min_seconds > 0.0:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(3):
            step()
        e1.record()
        torch.cuda.synchronize()
        est_ms = max_over_ranks([e0.elapsed_time(e1) / 3.0], dist, device)[0]
        steps = max(steps, int(min_seconds * 1e3 / est_ms * 0.98) + 1)   # a step in a long run is a little slower than est
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)] for _ in range(steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(device.index if device.index is not None else 0) if sample_clocks else None
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    t_start.record()
    for s in range(steps):
        step(evs[s])
    t_end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    if dist is not None:
        dist.barrier()
    total_ms = t_start.elapsed_time(t_end)
    per_call = {}
    for i, name in enumerate(calls):
        per_call[name] = sum(evs[s][i].elapsed_time(evs[s][i + 1]) for s in range(steps)) / steps
    if B.moe_device_status() != 0:
        raise RuntimeError("device status word is set after the timed region")
    return dict(wl=wl, buffers=b, total_ms=total_ms, per_call_ms=per_call, clocks=clocks, steps=steps)


def time_permute_alone(B, device, names, reps=15):
    """`moe_permute` outside the step, the way a data-movement kernel is usually judged: the chip idle for two seconds
    first (boost clocks, no power cap), L2 flushed before every call (a 256 MiB fill), median of `reps` calls, per
    workload.  Inside a step the same call runs at the SM clock the power cap leaves after a GEMM (per-call figures of
    the step, `stream_calibration_in_step`)."""
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    out = {}
    time.sleep(2.0)
    for name in names:
        cfg = W.CONFIGS[name]
        idx, _ = W.make_routing(cfg)
        idx = torch.from_numpy(idx).to(device)
        x = torch.randn(cfg.T, cfg.H, device=device).to(torch.bfloat16)
        d = B.dims(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K)
        xp = torch.empty((cfg.R, cfg.H), dtype=torch.bfloat16, device=device)
        i32 = lambda n: torch.empty(n, dtype=torch.int32, device=device)
        counts, offsets, r2p, p2r = i32(cfg.E), i32(cfg.E + 1), i32(cfg.R), i32(cfg.R)
        ws = torch.empty(max(B.moe_permute_workspace_bytes(d), 16), dtype=torch.uint8, device=device)
        call = lambda: B.moe_permute(d, x, idx, xp, counts, offsets, r2p, p2r, ws)
        for _ in range(3):
            call()
        times = []
        for _ in range(reps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            call()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = statistics.median(times)
        gbs = call_bytes(cfg)["permute"] / (ms * 1e-3) / 1e9
        out[name] = {"us": ms * 1e3, "gbs": gbs, "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS}
        del x, xp, idx
        torch.cuda.empty_cache()
    if B.moe_device_status() != 0:
        raise RuntimeError("device status word is set after the isolated permute calls")
    return out


def time_router(B, cfg, device, reps=30):
    """The router in front of the layer (outside the step the headline metric times): logits of the workload's own
    draw -> top-k indices and weights, and the backward to the logits.  Timed alone with CUDA events after
    3 warm-ups; the logits of the benchmark workloads are a few MB, so this measures launch plus a few microseconds."""
    if cfg.routing not in ("softmax", "skew"):
        return None
    z = torch.from_numpy(W.make_router_logits(cfg)).to(device)
    d = B.dims(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K)
    idx = torch.empty((cfg.T, cfg.K), dtype=torch.int32, device=device)
    w = torch.empty((cfg.T, cfg.K), dtype=torch.float32, device=device)
    dw = torch.randn((cfg.T, cfg.K), dtype=torch.float32, device=device)
    dz = torch.empty_like(z)
    out = {}
    for name, fn in (("fwd", lambda: B.moe_router_topk(d, z, idx, w)), ("bwd", lambda: B.moe_router_topk_bwd(d, idx, w, dw, dz))):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        out[name + "_ms"] = e0.elapsed_time(e1) / reps
    nbytes = cfg.T * cfg.E * 4 + cfg.T * cfg.K * 8
    out["fwd_gbs"] = nbytes / (out["fwd_ms"] * 1e-3) / 1e9
    out["bwd_gbs"] = (cfg.T * cfg.E * 4 + cfg.T * cfg.K * 12) / (out["bwd_ms"] * 1e-3) / 1e9
    out["note"] = "back-to-back launches, inputs L2-resident at these sizes"
    return out


def time_sustained(B, cfg, res, device, seconds=2.0):
    """The same step run back to back for at least `seconds` (the way the measured cuBLAS sustained peak was
    taken), so that the power and thermal state of a long run shows: steps in batches of 20 between two events."""
    step = make_step(B, res["buffers"], res["wl"])
    sampler = ClockSampler(device.index if device.index is not None else 0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    done, ms = 0, 0.0
    while ms < seconds * 1e3 and done < 200000:
        e0.record()
        for _ in range(20):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms += e0.elapsed_time(e1)
        done += 20
    clocks = sampler.stop()
    return {"seconds": ms * 1e-3, "steps": done, "ms_per_step": ms / done,
            "value": cfg.flops_fwd_bwd / (ms / done * 1e-3) / 1e12, "unit": UNIT, "clocks": clocks}


def fractions(tflops, peaks):
    """A tensor-bound rate against the three ceilings in use: nominal dense bf16, measured cuBLAS burst, measured
    cuBLAS sustained."""
    return {"of_nominal_2250": tflops / NOMINAL_BF16_TFLOPS, "of_measured_burst": tflops / peaks["bf16_tflops"],
            "of_measured_sustained": tflops / peaks["bf16_tflops_sustained"]}


def summarize(cfg, res, peaks, peaks_kind, sms):
    steps = res["steps"]
    ms_step = res["total_ms"] / steps
    pc = res["per_call_ms"]
    flops = call_flops(cfg)
    nbytes = call_bytes(cfg)
    gemm_ms = sum(pc[c] for c in GEMM_CALLS)
    gemm_tflops = cfg.flops_fwd_bwd / (gemm_ms * 1e-3) / 1e12
    mhz = (res["clocks"] or {}).get("sm_mhz")
    out = {
        "workload": cfg.name, "steps": steps, "timed_seconds": res["total_ms"] * 1e-3, "ms_per_step": ms_step,
        "layer_tflops": cfg.flops_fwd_bwd / (ms_step * 1e-3) / 1e12,
        "gemm_tflops": gemm_tflops,
        "gemm_frac": fractions(gemm_tflops, peaks),
        "per_call_ms": {k: round(v, 5) for k, v in pc.items()},
        "per_call_tflops": {c: round(flops[c] / (pc[c] * 1e-3) / 1e12, 1) for c in GEMM_CALLS},
        "per_call_gbs": {c: round(nbytes[c] / (pc[c] * 1e-3) / 1e9, 1) for c in nbytes},
        "per_call_gbs_frac_of_measured_copy": {c: round(nbytes[c] / (pc[c] * 1e-3) / 1e9 / peaks["hbm_gbs"], 3) for c in nbytes},
        "permute_gbs": nbytes["permute"] / (pc["permute"] * 1e-3) / 1e9,
        "permute_frac_of_nominal_8000": nbytes["permute"] / (pc["permute"] * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "permute_frac_of_measured": nbytes["permute"] / (pc["permute"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "roofline": roofline_object(cfg, res, peaks, peaks_kind),
        "clocks": res["clocks"],
    }
    if mhz:
        # clock-normalised: per-call time x the median SM clock sampled over these steps (millions of SM cycles), and
        # for the GEMMs the share of the tensor pipe's rate at that clock -- comparable across differently
        # power-capped boxes
        out["clock_normalised"] = {
            "sm_mhz_median": mhz,
            "per_call_mcycles": {k: round(v * 1e-3 * mhz, 3) for k, v in pc.items()},
            "per_call_pipe_frac_at_sampled_clock": {
                c: round(flops[c] / (pc[c] * 1e-3 * mhz * 1e6 * sms * PIPE_FLOP_PER_CLK_PER_SM), 3) for c in GEMM_CALLS},
            "gemm_pipe_frac_at_sampled_clock": cfg.flops_fwd_bwd / (gemm_ms * 1e-3 * mhz * 1e6 * sms * PIPE_FLOP_PER_CLK_PER_SM),
        }
    return out


def roofline_object(cfg, res, peaks, peaks_kind):
    """The grouped-GEMM call with the largest share of the step: algorithmic flops per launch / its average
    CUDA-event duration inside the timed steps, against the measured cuBLAS bf16 rates and the nominal peak."""
    pc = res["per_call_ms"]
    flops = call_flops(cfg)
    dom = max(GEMM_CALLS, key=lambda c: pc[c])
    achieved = flops[dom] / (pc[dom] * 1e-3) / 1e12
    # a run of a second or more sits under the power cap: the sustained cuBLAS rate is the like-for-like ceiling
    long_run = res["total_ms"] >= 1000.0
    peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
    traffic = NCU_TRAFFIC.get((cfg.name, dom))
    return {"bound": "tensor", "kernel": "grouped_gemm_kernel[" + dom + "]", "achieved": achieved, "peak": peak,
            "peak_kind": ("bf16 cuBLAS sustained (timed region >= 1 s), of " if long_run else "bf16 cuBLAS burst, of ") + peaks_kind,
            "unit": "TFLOP/s", "frac": achieved / peak,
            "frac_of_burst": achieved / peaks["bf16_tflops"], "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
            "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
            "flops_per_launch": flops[dom], "avg_launch_ms": pc[dom],
            "traffic": traffic[0] if traffic else None, "traffic_source": traffic[1] if traffic else None}


# --------------------------------------------------------------------------------------------
# end to end through the host-buffer entry point
# --------------------------------------------------------------------------------------------
def time_e2e(B, cfg, wl, b, device, steps, warmup, dist=None):
    """`steps` calls of moe_layer_fwd_bwd_host back to back: every call copies that step's activations, routing and
    upstream gradient from pinned host memory and copies y, dx and dtopk_w back to pinned host memory."""
    d = b.d
    arena = torch.empty(B.moe_layer_arena_bytes(d), dtype=torch.uint8, device=device)
    pin = lambda t: t.cpu().pin_memory()
    xh, ih, wh, dyh = pin(wl["X"]), pin(wl["topk_idx"]), pin(wl["topk_w"]), pin(wl["dY"])
    yh = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16).pin_memory()
    dxh = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16).pin_memory()
    dwh = torch.empty((cfg.T, cfg.K), dtype=torch.float32).pin_memory()

    def step():
        B.moe_layer_fwd_bwd_host(d, xh, ih, wh, dyh, wl["W_gate"], wl["W_up"], wl["W_down"], yh, dxh, dwh,
                                 b.dw_gate, b.dw_up, b.dw_down, arena)

    for _ in range(warmup):
        step()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    # the results that came back are the device-resident step's (same inputs, same kernels): bit for bit
    same = bool(torch.equal(yh, b.y.cpu()) and torch.equal(dxh, b.dx.cpu()))
    h2d = xh.numel() * 2 + ih.numel() * 4 + wh.numel() * 4 + dyh.numel() * 2
    d2h = yh.numel() * 2 + dxh.numel() * 2 + dwh.numel() * 4
    del arena
    return ms, h2d, d2h, same


# --------------------------------------------------------------------------------------------
# the fp64 oracle on the host cores (baseline, not the target)
# --------------------------------------------------------------------------------------------
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_time(host, cfg, n_tokens):
    """Runs the whole oracle chain on the first n_tokens tokens (all experts' weights); seconds."""
    from oracle import moe_oracle as O
    t0 = time.perf_counter()
    O.layer_fwd_bwd(host["X"][:n_tokens], host["topk_idx"][:n_tokens], host["topk_w"][:n_tokens], host["W_gate"],
                    host["W_up"], host["W_down"], host["dY"][:n_tokens])
    return time.perf_counter() - t0


def host_copy(wl):
    return {k: (v.to(torch.float32).cpu().numpy() if v.dtype == torch.bfloat16 else v.cpu().numpy())
            for k, v in wl.items()}


def cpu_baseline(cfg, host, n_tokens):
    oracle_sample_time(host, cfg, min(n_tokens, 16))          # first-touch / BLAS thread start-up, untimed
    sec = oracle_sample_time(host, cfg, n_tokens)
    fl = 18.0 * n_tokens * cfg.K * cfg.H * cfg.I
    return {"value": fl / sec / 1e12, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "sample": f"fp64 numpy oracle, whole fwd+bwd chain on the first {n_tokens} of {cfg.T} tokens of "
                      f"'{cfg.name}' (all {cfg.E} experts' weights), {sec:.1f} s",
            "seconds": sec}


# --------------------------------------------------------------------------------------------
def run_reference(args):
    """The oracle as the reference arm: rank 0 only, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = W.CONFIGS[args.config]
    host = W.make_workload(cfg) if args.host_inputs == "numpy" else None
    if host is None:
        if torch.cuda.is_available():
            host = host_copy(W.make_workload_device(cfg, torch.device("cuda", 0)))
        else:
            host = W.make_workload(cfg)
    n_tok = min(args.ref_tokens, cfg.T)
    budget = 240.0 / max(1, args.steps + args.warmup)
    oracle_sample_time(host, cfg, 16)
    while True:
        t = oracle_sample_time(host, cfg, n_tok)
        if t <= budget or n_tok <= 16:
            break
        n_tok //= 2
    for _ in range(max(0, args.warmup - 1)):
        oracle_sample_time(host, cfg, n_tok)
    times = [oracle_sample_time(host, cfg, n_tok) for _ in range(args.steps)]
    sec = sum(times) / len(times)
    value = 18.0 * n_tok * cfg.K * cfg.H * cfg.I / sec / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "I": cfg.I, "E": cfg.E, "K": cfg.K,
                       "sample_tokens_per_step": n_tok},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                             "sample": f"each step = fp64 numpy oracle fwd+bwd chain on the first {n_tok} of {cfg.T} tokens"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def stream_calibration(device):
    """Read-only, write-only and copy stream rates of this GPU right now (torch library kernels on a 2 GiB
    buffer).  Context for the data-movement kernels: their traffic mixes reads and writes very unevenly and
    the write-only rate of this part is far below its copy rate."""
    n = 1 << 30
    a = torch.empty(n, dtype=torch.bfloat16, device=device)
    b = torch.empty(n, dtype=torch.bfloat16, device=device)
    a.zero_()

    def rate(fn, nbytes, reps=10):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return nbytes * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9

    out = {"write_only_gbs": rate(lambda: a.fill_(1.0), 2 * n), "read_only_gbs": rate(lambda: a.sum(), 2 * n),
           "copy_gbs": rate(lambda: b.copy_(a), 4 * n)}
    del a, b
    torch.cuda.empty_cache()
    return out


def stream_calibration_in_step(B, cfg, res, device, steps=12):
    """The same three library stream kernels (512 MiB buffers), each timed with events right after a whole layer
    step, i.e. in the power-capped state the step's own data-movement kernels run in.  On this part the write-heavy
    rates drop well below their idle-chip values in that state while the read rate does not: context for the
    per-call GB/s of the write-heavy calls (permute, combine backward, SwiGLU backward)."""
    step = make_step(B, res["buffers"], res["wl"])
    n = 1 << 28
    a = torch.empty(n, dtype=torch.bfloat16, device=device)
    b = torch.empty(n, dtype=torch.bfloat16, device=device)
    a.zero_()
    kinds = {"copy_gbs": (lambda: b.copy_(a), 4 * n), "write_only_gbs": (lambda: a.fill_(1.0), 2 * n),
             "read_only_gbs": (lambda: a.sum(), 2 * n)}
    for _ in range(3):
        step()
    out = {}
    for name, (fn, nbytes) in kinds.items():
        evs = []
        for _ in range(steps):
            step()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        out[name] = nbytes / (statistics.median(x.elapsed_time(y) for x, y in evs) * 1e-3) / 1e9
    out["note"] = "torch copy_/fill_/sum on 512 MiB, each timed directly after a whole step of '" + cfg.name + "' (median)"
    del a, b
    torch.cuda.empty_cache()
    return out


def gemm_calibration(device, seconds=1.5):
    """The library bf16 GEMM (torch.matmul, 8192^3) on THIS box, the way the measured peaks were taken: best of 10 single
    calls (burst) and back to back for `seconds` with the SM clock sampled (sustained).  Boxes of the pool differ in how
    hard the power cap bites; this puts the layer's numbers and the library's on the same chip and in the same minute."""
    n = 8192
    a = torch.randn(n, n, device=device, dtype=torch.bfloat16)
    b = torch.randn(n, n, device=device, dtype=torch.bfloat16)
    c = torch.empty(n, n, device=device, dtype=torch.bfloat16)
    fl = 2.0 * n ** 3
    for _ in range(3):
        torch.matmul(a, b, out=c)
    best = float("inf")
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    sampler = ClockSampler(device.index if device.index is not None else 0)
    sampler.start()
    done, ms = 0, 0.0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    while ms < seconds * 1e3:
        e0.record()
        for _ in range(50):
            torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize()
        ms += e0.elapsed_time(e1)
        done += 50
    clocks = sampler.stop()
    del a, b, c
    torch.cuda.empty_cache()
    sustained = fl * done / (ms * 1e-3) / 1e12
    out = {"burst_tflops": fl / (best * 1e-3) / 1e12, "sustained_tflops": sustained, "clocks": clocks}
    if clocks.get("sm_mhz"):
        out["sustained_pipe_frac_at_sampled_clock"] = sustained * 1e12 / (clocks["sm_mhz"] * 1e6 * torch.cuda.get_device_properties(device).multi_processor_count * PIPE_FLOP_PER_CLK_PER_SM)
    return out


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def aggregate_tflops(world, flops_per_replica, ms_per_step):
    """Whole-job throughput of `world` independent replicas that all finished within ms_per_step."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


def run_ours(args):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback of the CUDA path)")
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group(backend="nccl", device_id=device)
        dist = dist_mod
    peaks, peaks_kind = load_peaks()
    cfg = W.CONFIGS[args.config]
    sms = torch.cuda.get_device_properties(device).multi_processor_count

    if args.only_steps:
        # profiling runs: the warm-up and the timed steps and nothing else (optionally the fused step form and the
        # block-scaled FP8 calls), one short line
        res = time_config(B, cfg, device, args.steps, args.warmup, dist, min_seconds=0.0, fused=args.fused)
        out = {"workload": cfg.name, "steps": res["steps"], "ms_per_step": res["total_ms"] / res["steps"],
               "per_call_ms": {k: round(v, 5) for k, v in res["per_call_ms"].items()}}
        if args.with_mxfp8:
            out["mxfp8"] = time_mxfp8(B, cfg, res, device, reps=1, min_seconds=0.0, warm=0)
            if args.fp8_step:
                out["fp8_step"] = time_fp8_step(B, cfg, res, device, min_seconds=0.3)
        print(json.dumps(out), flush=True)
        return
    res = time_config(B, cfg, device, args.steps, args.warmup, dist, min_seconds=args.min_seconds)
    steps = res["steps"]
    if args.no_e2e:
        e2e_ms, h2d, d2h, e2e_same = float("nan"), 0, 0, None
    else:
        e2e_ms, h2d, d2h, e2e_same = time_e2e(B, cfg, res["wl"], res["buffers"], device, steps, args.warmup, dist)

    total_ms, e2e_ms_max = max_over_ranks([res["total_ms"], e2e_ms], dist, device)
    ms_step = total_ms / steps
    value = aggregate_tflops(world, cfg.flops_fwd_bwd, ms_step)
    summary = summarize(cfg, res, peaks, peaks_kind, sms)
    launches_per_step = sum(LAUNCHES_PER_CALL.get(c, 1) for c in CALLS)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "steps_requested": args.steps,
        "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "I": cfg.I, "E": cfg.E, "K": cfg.K,
                   "routing": cfg.routing, "parallelism": "replicas only (single-GPU layer)" if world > 1 else "1 GPU",
                   "timed_seconds": total_ms * 1e-3,
                   "l2": "no flush: the step's working set (weights + activations) exceeds the 126 MB L2 many times"},
        "clocks": res["clocks"],
        "e2e": {"value": aggregate_tflops(world, cfg.flops_fwd_bwd, e2e_ms_max), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms_max,
                "results_equal_device_resident_step": e2e_same,
                "note": "moe_layer_fwd_bwd_host: activations, routing and upstream gradient from pinned host "
                        "memory each step, results read back each step; weights and weight gradients stay on the "
                        "device; the copies run on side streams and, with steps following one another, under the "
                        "neighbouring steps' GEMMs"},
        "gpu_launches": launches_per_step * steps,
        "roofline": summary["roofline"],
        "pct_of_dense_bf16_peak_nominal": 100.0 * summary["gemm_frac"]["of_nominal_2250"],
        "gemm_tflops": summary["gemm_tflops"], "permute_gbs": summary["permute_gbs"],
        "detail": summary, "peaks": {"kind": peaks_kind, "hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks["bf16_tflops"],
                                     "bf16_tflops_sustained": peaks["bf16_tflops_sustained"],
                                     "nominal_bf16_tflops": NOMINAL_BF16_TFLOPS, "nominal_hbm_gbs": NOMINAL_HBM_GBS},
    }

    if rank == 0 and world == 1:
        extra = []
        wl_host = None
        if not args.no_cpu_baseline:
            n_tok = min(args.ref_tokens, cfg.T)
            wl_host = host_copy({k: (v[:n_tok] if k in ("X", "dY", "topk_idx", "topk_w") else v) for k, v in res["wl"].items()})
        line["sustained"] = time_sustained(B, cfg, res, device)
        line["sustained"]["frac"] = fractions(line["sustained"]["value"], peaks)
        line["stream_calibration_in_step"] = stream_calibration_in_step(B, cfg, res, device)
        line["fused_dgrad_swiglu_bwd"] = time_fused_variant(B, cfg, res, device)
        line["mxfp8"] = time_mxfp8(B, cfg, res, device)
        line["fp8_step"] = time_fp8_step(B, cfg, res, device)
        del res
        torch.cuda.empty_cache()
        for name in args.also:
            if name == cfg.name:
                continue
            c2 = W.CONFIGS[name]
            r2 = time_config(B, c2, device, 3, 3, None, sample_clocks=True, min_seconds=args.other_min_seconds)
            extra.append(summarize(c2, r2, peaks, peaks_kind, sms))
            extra[-1]["fused_dgrad_swiglu_bwd"] = time_fused_variant(B, c2, r2, device, seconds=0.5)
            extra[-1]["mxfp8"] = time_mxfp8(B, c2, r2, device)
            extra[-1]["fp8_step"] = time_fp8_step(B, c2, r2, device, min_seconds=0.3)
            del r2
            torch.cuda.empty_cache()
        if extra:
            line["other_configs"] = extra
        router_cfg = cfg if cfg.routing in ("softmax", "skew") else W.CONFIGS["many_small"]
        router = time_router(B, router_cfg, device)
        if router is not None:
            router["workload"] = router_cfg.name
            line["router"] = router
        line["permute_alone"] = time_permute_alone(B, device, [cfg.name] + [n for n in args.also if n != cfg.name])
        line["stream_calibration"] = stream_calibration(device)
        line["gemm_calibration"] = gemm_calibration(device)
        if wl_host is not None:
            line["cpu_baseline"] = cpu_baseline(cfg, wl_host, min(args.ref_tokens, cfg.T))
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", default="imbalanced", choices=list(W.CONFIGS))
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="the headline workload's timed region lasts at least this long (steps are added to --steps)")
    ap.add_argument("--other-min-seconds", type=float, default=0.5, help="the same floor for each of the --also workloads")
    ap.add_argument("--custom", default="", help="T,H,I,E,K of an ad-hoc softmax-routed workload (profiling aid)")
    ap.add_argument("--scale", type=int, default=1,
                    help="profiling aid: run a 1/SCALE copy of --config (tokens and experts divided by SCALE; same H, I, "
                         "top-k, routing law and rows per expert) so that a multi-pass ncu capture stays small")
    ap.add_argument("--also", default="fine_grained,many_small,few_large,paper_dw1",
                    help="comma-separated other configurations to time briefly at N=1 ('' for none)")
    ap.add_argument("--ref-tokens", type=int, default=1024, help="tokens in the oracle's timed sample")
    ap.add_argument("--host-inputs", default="device", choices=["device", "numpy"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer pass (profiling runs)")
    ap.add_argument("--only-steps", action="store_true", help="profiling runs: warm-up and timed steps only")
    ap.add_argument("--fused", action="store_true", help="with --only-steps: the step form with the fused down-dgrad + SwiGLU-backward call")
    ap.add_argument("--with-mxfp8", action="store_true", help="with --only-steps: also run the block-scaled FP8 calls")
    ap.add_argument("--fp8-step", action="store_true", help="with --only-steps --with-mxfp8: also time the FP8 form of the step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    args.also = [s for s in args.also.split(",") if s]
    if args.custom:
        T, H, I, E, K = (int(v) for v in args.custom.split(","))
        W.CONFIGS["custom"] = W.MoeConfig("custom", T=T, H=H, I=I, E=E, K=K, routing="softmax", cfg_id=9)
        args.config = "custom"
    if args.scale > 1:
        c = W.CONFIGS[args.config]
        name = f"{c.name}_scaled{args.scale}"
        W.CONFIGS[name] = W.MoeConfig(name, T=c.T // args.scale, H=c.H, I=c.I, E=c.E // args.scale, K=c.K, routing=c.routing,
                                      n_empty=max(1, c.n_empty // args.scale) if c.n_empty else 0, cfg_id=c.cfg_id)
        args.config = name
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
