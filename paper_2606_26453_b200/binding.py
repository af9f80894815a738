"""Thin ctypes binding over libmoe_b200.so: argument marshalling only.

Every function has the name and argument order of its C entry point (include/moe_b200.h) and takes
torch CUDA tensors (used purely as device memory) plus the current torch stream.  Nothing is
computed here; a missing library or a non-zero status raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libmoe_b200.so")

EXPORTS = [
    "moe_status_string", "moe_permute_workspace_bytes", "moe_device_status", "moe_permute", "moe_permute_static_scratch",
    "moe_permute_bwd",
    "moe_grouped_gemm_gateup_swiglu", "moe_grouped_gemm_down", "moe_unpermute_combine",
    "moe_unpermute_combine_bwd", "moe_grouped_gemm_down_dgrad", "moe_grouped_gemm_down_wgrad",
    "moe_grouped_gemm_down_bwd", "moe_swiglu_bwd", "moe_grouped_gemm_down_dgrad_swiglu_bwd", "moe_grouped_gemm_gateup_dgrad",
    "moe_grouped_gemm_gateup_wgrad", "moe_grouped_gemm_gateup_swiglu_bwd", "moe_layer_arena_bytes",
    "moe_layer_fwd_bwd_host", "moe_router_topk", "moe_router_topk_bwd",
    "moe_mxfp8_act_scale_bytes", "moe_mxfp8_w_down_scale_bytes", "moe_mxfp8_quantize_h_act", "moe_mxfp8_quantize_w_down",
    "moe_grouped_gemm_down_mxfp8",
    "moe_mxfp8_dy_scale_bytes", "moe_mxfp8_w_down_dgrad_scale_bytes", "moe_mxfp8_quantize_dy_perm",
    "moe_mxfp8_quantize_w_down_dgrad", "moe_grouped_gemm_down_dgrad_mxfp8",
    "moe_mxfp8_dgu_scale_bytes", "moe_mxfp8_w_gateup_dgrad_scale_bytes", "moe_mxfp8_quantize_dgu",
    "moe_mxfp8_quantize_w_gateup_dgrad", "moe_grouped_gemm_gateup_dgrad_mxfp8",
    "moe_mxfp8_x_scale_bytes", "moe_mxfp8_w_gateup_scale_bytes", "moe_mxfp8_quantize_x_perm", "moe_mxfp8_quantize_w_gateup",
    "moe_grouped_gemm_gateup_mxfp8", "moe_swiglu_mxfp8",
    "moe_mxfp8_tokens_codes_bytes", "moe_mxfp8_tokens_scale_bytes", "moe_mxfp8_quantize_tokens",
    "moe_grouped_gemm_down_wgrad_mxfp8", "moe_grouped_gemm_gateup_wgrad_mxfp8", "moe_swiglu_bwd_mxfp8",
]


class MoeDims(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("H", ctypes.c_int32), ("I", ctypes.c_int32), ("E", ctypes.c_int32),
                ("K", ctypes.c_int32)]


class MoeError(RuntimeError):
    def __init__(self, fn: str, status: int, text: str):
        super().__init__(f"{fn} failed: status {status} ({text})")
        self.status = status


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2606_26453_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        lib.moe_status_string.restype = ctypes.c_char_p
        lib.moe_status_string.argtypes = [ctypes.c_int]
        lib.moe_permute_workspace_bytes.restype = ctypes.c_size_t
        lib.moe_permute_workspace_bytes.argtypes = [ctypes.POINTER(MoeDims)]
        lib.moe_layer_arena_bytes.restype = ctypes.c_size_t
        lib.moe_layer_arena_bytes.argtypes = [ctypes.POINTER(MoeDims)]
        for name in ("moe_mxfp8_act_scale_bytes", "moe_mxfp8_w_down_scale_bytes", "moe_mxfp8_dy_scale_bytes",
                     "moe_mxfp8_w_down_dgrad_scale_bytes", "moe_mxfp8_dgu_scale_bytes",
                     "moe_mxfp8_w_gateup_dgrad_scale_bytes", "moe_mxfp8_x_scale_bytes", "moe_mxfp8_w_gateup_scale_bytes"):
            getattr(lib, name).restype = ctypes.c_size_t
            getattr(lib, name).argtypes = [ctypes.POINTER(MoeDims)]
        for name in ("moe_mxfp8_tokens_codes_bytes", "moe_mxfp8_tokens_scale_bytes"):
            getattr(lib, name).restype = ctypes.c_size_t
            getattr(lib, name).argtypes = [ctypes.POINTER(MoeDims), ctypes.c_int]
        lib.moe_device_status.restype = ctypes.c_int
        lib.moe_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
        p = ctypes.c_void_p
        dp = ctypes.POINTER(MoeDims)
        sigs = {
            "moe_permute": [dp, p, p, p, p, p, p, p, p, ctypes.c_size_t, p],
            "moe_permute_static_scratch": [dp, p, p, p, p, p, p, p, p],
            "moe_permute_bwd": [dp, p, p, p, p],
            "moe_grouped_gemm_gateup_swiglu": [dp, p, p, p, p, p, p, p],
            "moe_grouped_gemm_down": [dp, p, p, p, p, p],
            "moe_unpermute_combine": [dp, p, p, p, p, p],
            "moe_unpermute_combine_bwd": [dp, p, p, p, p, p, p, p],
            "moe_grouped_gemm_down_dgrad": [dp, p, p, p, p, p],
            "moe_grouped_gemm_down_wgrad": [dp, p, p, p, p, p],
            "moe_grouped_gemm_down_bwd": [dp, p, p, p, p, p, p, p],
            "moe_swiglu_bwd": [dp, p, p, p, p],
            "moe_grouped_gemm_down_dgrad_swiglu_bwd": [dp, p, p, p, p, p, p],
            "moe_router_topk": [dp, p, p, p, p],
            "moe_router_topk_bwd": [dp, p, p, p, p, p],
            "moe_grouped_gemm_gateup_dgrad": [dp, p, p, p, p, p, p],
            "moe_grouped_gemm_gateup_wgrad": [dp, p, p, p, p, p, p],
            "moe_grouped_gemm_gateup_swiglu_bwd": [dp, p, p, p, p, p, p, p, p, p, p, p],
            "moe_layer_fwd_bwd_host": [dp] + [p] * 14 + [ctypes.c_size_t, p],
            "moe_mxfp8_quantize_h_act": [dp, p, p, p, p],
            "moe_mxfp8_quantize_w_down": [dp, p, p, p, p],
            "moe_grouped_gemm_down_mxfp8": [dp, p, p, p, p, p, p, p],
            "moe_mxfp8_quantize_dy_perm": [dp, p, p, p, p],
            "moe_mxfp8_quantize_w_down_dgrad": [dp, p, p, p, p],
            "moe_grouped_gemm_down_dgrad_mxfp8": [dp, p, p, p, p, p, p, p],
            "moe_mxfp8_quantize_dgu": [dp, p, p, p, p],
            "moe_mxfp8_quantize_w_gateup_dgrad": [dp, p, p, p, p, p],
            "moe_grouped_gemm_gateup_dgrad_mxfp8": [dp, p, p, p, p, p, p, p],
            "moe_mxfp8_quantize_x_perm": [dp, p, p, p, p],
            "moe_mxfp8_quantize_w_gateup": [dp, p, p, p, p, p],
            "moe_grouped_gemm_gateup_mxfp8": [dp, p, p, p, p, p, p, p],
            "moe_swiglu_mxfp8": [dp, p, p, p, p, p],
            "moe_swiglu_bwd_mxfp8": [dp, p, p, p, p, p, p],
            "moe_mxfp8_quantize_tokens": [dp, p, ctypes.c_int, ctypes.c_int, ctypes.c_int, p, p, p, p],
            "moe_grouped_gemm_down_wgrad_mxfp8": [dp, p, p, p, p, p, p],
            "moe_grouped_gemm_gateup_wgrad_mxfp8": [dp, p, p, p, p, p, p, p, p, p],
        }
        for name, argtypes in sigs.items():
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = argtypes
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().moe_status_string(int(status)).decode()


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _call(name: str, *args) -> None:
    rc = getattr(load_library(), name)(*args)
    if rc != 0:
        raise MoeError(name, rc, status_string(rc))


def dims(T: int, H: int, I: int, E: int, K: int) -> MoeDims:
    return MoeDims(T, H, I, E, K)


def moe_permute_workspace_bytes(d: MoeDims) -> int:
    return int(load_library().moe_permute_workspace_bytes(ctypes.byref(d)))


def moe_layer_arena_bytes(d: MoeDims) -> int:
    return int(load_library().moe_layer_arena_bytes(ctypes.byref(d)))


def moe_device_status() -> int:
    out = ctypes.c_int(0)
    rc = load_library().moe_device_status(ctypes.byref(out))
    if rc != 0:
        raise MoeError("moe_device_status", rc, status_string(rc))
    return out.value


def moe_permute(d, x, topk_idx, x_perm, counts, offsets, row_to_pair, pair_to_row, workspace):
    _call("moe_permute", ctypes.byref(d), _ptr(x), _ptr(topk_idx), _ptr(x_perm), _ptr(counts), _ptr(offsets),
          _ptr(row_to_pair), _ptr(pair_to_row), _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
          _stream())


def moe_permute_static_scratch(d, x, topk_idx, x_perm, counts, offsets, row_to_pair, pair_to_row):
    """moe_permute for callers that may not allocate: the scratch is a fixed array inside the library
    (shared by all calls on a device; see the header for the size limit and the no-overlap rule)."""
    _call("moe_permute_static_scratch", ctypes.byref(d), _ptr(x), _ptr(topk_idx), _ptr(x_perm), _ptr(counts),
          _ptr(offsets), _ptr(row_to_pair), _ptr(pair_to_row), _stream())


def moe_permute_bwd(d, dx_perm, pair_to_row, dx):
    _call("moe_permute_bwd", ctypes.byref(d), _ptr(dx_perm), _ptr(pair_to_row), _ptr(dx), _stream())


def moe_grouped_gemm_gateup_swiglu(d, x_perm, w_gate, w_up, offsets, h_act, gu_saved):
    _call("moe_grouped_gemm_gateup_swiglu", ctypes.byref(d), _ptr(x_perm), _ptr(w_gate), _ptr(w_up), _ptr(offsets),
          _ptr(h_act), _ptr(gu_saved), _stream())


def moe_grouped_gemm_down(d, h_act, w_down, offsets, y_perm):
    _call("moe_grouped_gemm_down", ctypes.byref(d), _ptr(h_act), _ptr(w_down), _ptr(offsets), _ptr(y_perm), _stream())


def moe_unpermute_combine(d, y_perm, topk_w, pair_to_row, y):
    _call("moe_unpermute_combine", ctypes.byref(d), _ptr(y_perm), _ptr(topk_w), _ptr(pair_to_row), _ptr(y), _stream())


def moe_unpermute_combine_bwd(d, dy, y_perm, topk_w, pair_to_row, dy_perm, dtopk_w):
    _call("moe_unpermute_combine_bwd", ctypes.byref(d), _ptr(dy), _ptr(y_perm), _ptr(topk_w), _ptr(pair_to_row),
          _ptr(dy_perm), _ptr(dtopk_w), _stream())


def moe_grouped_gemm_down_dgrad(d, dy_perm, w_down, offsets, dh_act):
    _call("moe_grouped_gemm_down_dgrad", ctypes.byref(d), _ptr(dy_perm), _ptr(w_down), _ptr(offsets), _ptr(dh_act),
          _stream())


def moe_grouped_gemm_down_wgrad(d, h_act, dy_perm, offsets, dw_down):
    _call("moe_grouped_gemm_down_wgrad", ctypes.byref(d), _ptr(h_act), _ptr(dy_perm), _ptr(offsets), _ptr(dw_down),
          _stream())


def moe_grouped_gemm_down_bwd(d, dy_perm, h_act, w_down, offsets, dh_act, dw_down):
    _call("moe_grouped_gemm_down_bwd", ctypes.byref(d), _ptr(dy_perm), _ptr(h_act), _ptr(w_down), _ptr(offsets),
          _ptr(dh_act), _ptr(dw_down), _stream())


def moe_router_topk(d, logits, topk_idx, topk_w):
    _call("moe_router_topk", ctypes.byref(d), _ptr(logits), _ptr(topk_idx), _ptr(topk_w), _stream())


def moe_router_topk_bwd(d, topk_idx, topk_w, dtopk_w, dlogits):
    _call("moe_router_topk_bwd", ctypes.byref(d), _ptr(topk_idx), _ptr(topk_w), _ptr(dtopk_w), _ptr(dlogits), _stream())


def moe_swiglu_bwd(d, dh_act, gu_saved, dgu):
    _call("moe_swiglu_bwd", ctypes.byref(d), _ptr(dh_act), _ptr(gu_saved), _ptr(dgu), _stream())


def moe_grouped_gemm_down_dgrad_swiglu_bwd(d, dy_perm, w_down, gu_saved, offsets, dgu):
    _call("moe_grouped_gemm_down_dgrad_swiglu_bwd", ctypes.byref(d), _ptr(dy_perm), _ptr(w_down), _ptr(gu_saved),
          _ptr(offsets), _ptr(dgu), _stream())


def moe_grouped_gemm_gateup_dgrad(d, dgu, w_gate, w_up, offsets, dx_perm):
    _call("moe_grouped_gemm_gateup_dgrad", ctypes.byref(d), _ptr(dgu), _ptr(w_gate), _ptr(w_up), _ptr(offsets),
          _ptr(dx_perm), _stream())


def moe_grouped_gemm_gateup_wgrad(d, x_perm, dgu, offsets, dw_gate, dw_up):
    _call("moe_grouped_gemm_gateup_wgrad", ctypes.byref(d), _ptr(x_perm), _ptr(dgu), _ptr(offsets), _ptr(dw_gate),
          _ptr(dw_up), _stream())


def moe_grouped_gemm_gateup_swiglu_bwd(d, dh_act, gu_saved, x_perm, w_gate, w_up, offsets, dgu, dx_perm, dw_gate, dw_up):
    _call("moe_grouped_gemm_gateup_swiglu_bwd", ctypes.byref(d), _ptr(dh_act), _ptr(gu_saved), _ptr(x_perm),
          _ptr(w_gate), _ptr(w_up), _ptr(offsets), _ptr(dgu), _ptr(dx_perm), _ptr(dw_gate), _ptr(dw_up), _stream())


def moe_mxfp8_act_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_act_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_w_down_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_w_down_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_quantize_h_act(d, h_act, codes, scales):
    _call("moe_mxfp8_quantize_h_act", ctypes.byref(d), _ptr(h_act), _ptr(codes), _ptr(scales), _stream())


def moe_mxfp8_quantize_w_down(d, w_down, codes_t, scales):
    _call("moe_mxfp8_quantize_w_down", ctypes.byref(d), _ptr(w_down), _ptr(codes_t), _ptr(scales), _stream())


def moe_grouped_gemm_down_mxfp8(d, h_codes, h_scales, w_codes_t, w_scales, offsets, y_perm):
    _call("moe_grouped_gemm_down_mxfp8", ctypes.byref(d), _ptr(h_codes), _ptr(h_scales), _ptr(w_codes_t), _ptr(w_scales),
          _ptr(offsets), _ptr(y_perm), _stream())


def moe_mxfp8_dy_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_dy_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_w_down_dgrad_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_w_down_dgrad_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_quantize_dy_perm(d, dy_perm, codes, scales):
    _call("moe_mxfp8_quantize_dy_perm", ctypes.byref(d), _ptr(dy_perm), _ptr(codes), _ptr(scales), _stream())


def moe_mxfp8_quantize_w_down_dgrad(d, w_down, codes, scales):
    _call("moe_mxfp8_quantize_w_down_dgrad", ctypes.byref(d), _ptr(w_down), _ptr(codes), _ptr(scales), _stream())


def moe_grouped_gemm_down_dgrad_mxfp8(d, dy_codes, dy_scales, w_codes, w_scales, offsets, dh_act):
    _call("moe_grouped_gemm_down_dgrad_mxfp8", ctypes.byref(d), _ptr(dy_codes), _ptr(dy_scales), _ptr(w_codes), _ptr(w_scales),
          _ptr(offsets), _ptr(dh_act), _stream())


def moe_mxfp8_dgu_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_dgu_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_w_gateup_dgrad_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_w_gateup_dgrad_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_quantize_dgu(d, dgu, codes, scales):
    _call("moe_mxfp8_quantize_dgu", ctypes.byref(d), _ptr(dgu), _ptr(codes), _ptr(scales), _stream())


def moe_mxfp8_quantize_w_gateup_dgrad(d, w_gate, w_up, codes, scales):
    _call("moe_mxfp8_quantize_w_gateup_dgrad", ctypes.byref(d), _ptr(w_gate), _ptr(w_up), _ptr(codes), _ptr(scales), _stream())


def moe_grouped_gemm_gateup_dgrad_mxfp8(d, dgu_codes, dgu_scales, w_codes, w_scales, offsets, dx_perm):
    _call("moe_grouped_gemm_gateup_dgrad_mxfp8", ctypes.byref(d), _ptr(dgu_codes), _ptr(dgu_scales), _ptr(w_codes),
          _ptr(w_scales), _ptr(offsets), _ptr(dx_perm), _stream())


def moe_mxfp8_x_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_x_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_w_gateup_scale_bytes(d: MoeDims) -> int:
    return int(load_library().moe_mxfp8_w_gateup_scale_bytes(ctypes.byref(d)))


def moe_mxfp8_quantize_x_perm(d, x_perm, codes, scales):
    _call("moe_mxfp8_quantize_x_perm", ctypes.byref(d), _ptr(x_perm), _ptr(codes), _ptr(scales), _stream())


def moe_mxfp8_quantize_w_gateup(d, w_gate, w_up, codes_t, scales):
    _call("moe_mxfp8_quantize_w_gateup", ctypes.byref(d), _ptr(w_gate), _ptr(w_up), _ptr(codes_t), _ptr(scales), _stream())


def moe_grouped_gemm_gateup_mxfp8(d, x_codes, x_scales, w_codes_t, w_scales, offsets, gu):
    _call("moe_grouped_gemm_gateup_mxfp8", ctypes.byref(d), _ptr(x_codes), _ptr(x_scales), _ptr(w_codes_t), _ptr(w_scales),
          _ptr(offsets), _ptr(gu), _stream())


def moe_swiglu_mxfp8(d, gu, h_act, h_codes, h_scales):
    _call("moe_swiglu_mxfp8", ctypes.byref(d), _ptr(gu), _ptr(h_act), _ptr(h_codes), _ptr(h_scales), _stream())


def moe_mxfp8_tokens_codes_bytes(d: MoeDims, n_features: int) -> int:
    return int(load_library().moe_mxfp8_tokens_codes_bytes(ctypes.byref(d), int(n_features)))


def moe_mxfp8_tokens_scale_bytes(d: MoeDims, n_features: int) -> int:
    return int(load_library().moe_mxfp8_tokens_scale_bytes(ctypes.byref(d), int(n_features)))


def moe_mxfp8_quantize_tokens(d, x, ld, col0, n_features, offsets, codes_t, scales):
    _call("moe_mxfp8_quantize_tokens", ctypes.byref(d), _ptr(x), int(ld), int(col0), int(n_features), _ptr(offsets),
          _ptr(codes_t), _ptr(scales), _stream())


def moe_grouped_gemm_down_wgrad_mxfp8(d, h_codes_t, h_scales, dy_codes_t, dy_scales, dw_down):
    _call("moe_grouped_gemm_down_wgrad_mxfp8", ctypes.byref(d), _ptr(h_codes_t), _ptr(h_scales), _ptr(dy_codes_t),
          _ptr(dy_scales), _ptr(dw_down), _stream())


def moe_grouped_gemm_gateup_wgrad_mxfp8(d, x_codes_t, x_scales, dg_codes_t, dg_scales, du_codes_t, du_scales, dw_gate, dw_up):
    _call("moe_grouped_gemm_gateup_wgrad_mxfp8", ctypes.byref(d), _ptr(x_codes_t), _ptr(x_scales), _ptr(dg_codes_t),
          _ptr(dg_scales), _ptr(du_codes_t), _ptr(du_scales), _ptr(dw_gate), _ptr(dw_up), _stream())


def moe_swiglu_bwd_mxfp8(d, dh_act, gu_saved, dgu, dgu_codes, dgu_scales):
    _call("moe_swiglu_bwd_mxfp8", ctypes.byref(d), _ptr(dh_act), _ptr(gu_saved), _ptr(dgu), _ptr(dgu_codes), _ptr(dgu_scales),
          _stream())


def moe_layer_fwd_bwd_host(d, x_host, topk_idx_host, topk_w_host, dy_host, w_gate, w_up, w_down, y_host, dx_host,
                           dtopk_w_host, dw_gate, dw_up, dw_down, arena):
    """x_host, topk_idx_host, topk_w_host, dy_host, y_host, dx_host, dtopk_w_host are CPU tensors
    (pinned for asynchronous copies); the rest are CUDA tensors."""
    _call("moe_layer_fwd_bwd_host", ctypes.byref(d), _ptr(x_host), _ptr(topk_idx_host), _ptr(topk_w_host),
          _ptr(dy_host), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(y_host), _ptr(dx_host), _ptr(dtopk_w_host),
          _ptr(dw_gate), _ptr(dw_up), _ptr(dw_down), _ptr(arena),
          ctypes.c_size_t(arena.numel() * arena.element_size()), _stream())


# ---------------------------------------------------------------------------------------------
# Buffer bundle for one layer step (allocation only; every step of the path is a library call)
# ---------------------------------------------------------------------------------------------
@dataclass
class LayerBuffers:
    d: MoeDims
    x_perm: torch.Tensor
    counts: torch.Tensor
    offsets: torch.Tensor
    row_to_pair: torch.Tensor
    pair_to_row: torch.Tensor
    workspace: torch.Tensor
    h_act: torch.Tensor
    gu: torch.Tensor
    y_perm: torch.Tensor
    y: torch.Tensor
    dy_perm: torch.Tensor
    dtopk_w: torch.Tensor
    dh_act: torch.Tensor
    dw_down: torch.Tensor
    dgu: torch.Tensor
    dx_perm: torch.Tensor
    dw_gate: torch.Tensor
    dw_up: torch.Tensor
    dx: torch.Tensor


def alloc_layer_buffers(T, H, I, E, K, device="cuda") -> LayerBuffers:
    d = dims(T, H, I, E, K)
    R = T * K
    bf = dict(dtype=torch.bfloat16, device=device)
    i32 = dict(dtype=torch.int32, device=device)
    ws = max(moe_permute_workspace_bytes(d), 16)
    return LayerBuffers(
        d=d, x_perm=torch.empty((R, H), **bf), counts=torch.empty(E, **i32), offsets=torch.empty(E + 1, **i32),
        row_to_pair=torch.empty(R, **i32), pair_to_row=torch.empty(R, **i32),
        workspace=torch.empty(ws, dtype=torch.uint8, device=device),
        h_act=torch.empty((R, I), **bf), gu=torch.empty((R, 2 * I), **bf), y_perm=torch.empty((R, H), **bf),
        y=torch.empty((T, H), **bf), dy_perm=torch.empty((R, H), **bf),
        dtopk_w=torch.empty((T, K), dtype=torch.float32, device=device), dh_act=torch.empty((R, I), **bf),
        dw_down=torch.empty((E, I, H), **bf), dgu=torch.empty((R, 2 * I), **bf), dx_perm=torch.empty((R, H), **bf),
        dw_gate=torch.empty((E, H, I), **bf), dw_up=torch.empty((E, H, I), **bf), dx=torch.empty((T, H), **bf))


def layer_forward(b: LayerBuffers, x, topk_idx, topk_w, w_gate, w_up, w_down):
    """a1..a4 in order on the current stream."""
    moe_permute(b.d, x, topk_idx, b.x_perm, b.counts, b.offsets, b.row_to_pair, b.pair_to_row, b.workspace)
    moe_grouped_gemm_gateup_swiglu(b.d, b.x_perm, w_gate, w_up, b.offsets, b.h_act, b.gu)
    moe_grouped_gemm_down(b.d, b.h_act, w_down, b.offsets, b.y_perm)
    moe_unpermute_combine(b.d, b.y_perm, topk_w, b.pair_to_row, b.y)


def layer_backward(b: LayerBuffers, dy, topk_w, w_gate, w_up, w_down, fused_swiglu_bwd: bool = False):
    """a5..a8 in order on the current stream (after layer_forward).  With fused_swiglu_bwd the down dgrad and the
    SwiGLU backward run as the one fused call (dh_act is then not written)."""
    moe_unpermute_combine_bwd(b.d, dy, b.y_perm, topk_w, b.pair_to_row, b.dy_perm, b.dtopk_w)
    if fused_swiglu_bwd:
        moe_grouped_gemm_down_dgrad_swiglu_bwd(b.d, b.dy_perm, w_down, b.gu, b.offsets, b.dgu)
        moe_grouped_gemm_down_wgrad(b.d, b.h_act, b.dy_perm, b.offsets, b.dw_down)
        moe_grouped_gemm_gateup_dgrad(b.d, b.dgu, w_gate, w_up, b.offsets, b.dx_perm)
        moe_grouped_gemm_gateup_wgrad(b.d, b.x_perm, b.dgu, b.offsets, b.dw_gate, b.dw_up)
    else:
        moe_grouped_gemm_down_bwd(b.d, b.dy_perm, b.h_act, w_down, b.offsets, b.dh_act, b.dw_down)
        moe_grouped_gemm_gateup_swiglu_bwd(b.d, b.dh_act, b.gu, b.x_perm, w_gate, w_up, b.offsets, b.dgu, b.dx_perm,
                                           b.dw_gate, b.dw_up)
    moe_permute_bwd(b.d, b.dx_perm, b.pair_to_row, b.dx)
