"""Shared helpers of the GPU parity tests: tolerances, tensor conversion, running the CUDA path."""
from __future__ import annotations

import numpy as np
import torch

from paper_2606_26453_b200 import workloads as W

MAX_ABS_FACTOR = 2e-2     # max|err| <= 2e-2 * max|ref|
REL_FROBENIUS = 5e-3      # ||err||_F / ||ref||_F <= 5e-3
PER_CALL_FROBENIUS = 2.5e-3   # one bf16 rounding of an output gives ~1.7e-3; more means a bug


def to_dev_bf16(a: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device).to(torch.bfloat16)


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def error_stats(got: np.ndarray, ref: np.ndarray):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    err = got - ref
    max_ref = float(np.max(np.abs(ref))) if ref.size else 0.0
    nref = float(np.linalg.norm(ref))
    return dict(max_err=float(np.max(np.abs(err))) if err.size else 0.0, max_ref=max_ref,
                rel_fro=float(np.linalg.norm(err) / nref) if nref > 0 else (0.0 if not err.any() else np.inf))


def assert_close(got, ref, name, rel_fro=REL_FROBENIUS, max_abs=MAX_ABS_FACTOR):
    assert np.all(np.isfinite(got)), f"{name}: non-finite values in the CUDA result"
    s = error_stats(got, ref)
    if s["max_ref"] == 0.0:
        assert not np.any(got), f"{name}: reference is all zeros, result is not"
        return s
    assert s["max_err"] <= max_abs * s["max_ref"], f"{name}: max|err| {s['max_err']:.3e} > {max_abs} * {s['max_ref']:.3e}"
    assert s["rel_fro"] <= rel_fro, f"{name}: relative Frobenius error {s['rel_fro']:.3e} > {rel_fro}"
    return s


def device_workload(host: dict, device="cuda") -> dict:
    """Host workload (numpy, bf16-representable float32) -> torch tensors on the device."""
    out = {}
    for k, v in host.items():
        if k == "topk_idx":
            out[k] = torch.from_numpy(v).to(device)
        elif k == "topk_w":
            out[k] = torch.from_numpy(v).to(device)
        else:
            out[k] = to_dev_bf16(v, device)
    return out


def host_view(dev: dict) -> dict:
    """Device workload -> numpy arrays for the oracle (exact values)."""
    out = {}
    for k, v in dev.items():
        if v.dtype == torch.bfloat16:
            out[k] = v.to(torch.float32).cpu().numpy()
        else:
            out[k] = v.cpu().numpy()
    return out


def run_cuda_layer(dev: dict, E: int, fused_swiglu_bwd: bool = False):
    """Forward + backward through the C ABI; returns the buffer bundle."""
    from paper_2606_26453_b200 import binding as B
    T, H = dev["X"].shape
    K = dev["topk_idx"].shape[1]
    I = dev["W_gate"].shape[2]
    b = B.alloc_layer_buffers(T, H, I, E, K, device=dev["X"].device)
    B.layer_forward(b, dev["X"], dev["topk_idx"], dev["topk_w"], dev["W_gate"], dev["W_up"], dev["W_down"])
    B.layer_backward(b, dev["dY"], dev["topk_w"], dev["W_gate"], dev["W_up"], dev["W_down"],
                     fused_swiglu_bwd=fused_swiglu_bwd)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    return b


def ragged_workload(counts, K, H, I, seed=0):
    """Workload with prescribed per-expert row counts (host arrays)."""
    counts = np.asarray(counts)
    E = counts.size
    idx, w = W.make_routing_from_counts(counts, K, seed)
    T = idx.shape[0]
    cfg = W.MoeConfig("ragged", T=T, H=H, I=I, E=E, K=K, cfg_id=50 + seed)
    d = W.make_tensors(cfg, seed)
    d["topk_idx"], d["topk_w"] = idx, w
    return cfg, d
