"""The give-up path of the device-side waits, exercised without a fault: a test-only build of the library (waits
run out after 20 ms instead of 2 s) has a switch that makes every producer leave out the loads and the barrier
arrival of its first ring stage.  The MMA warp's wait on that stage then runs out: the kernel must come back by
itself, the device status word must read MOE_ERR_TIMEOUT, and the context must stay usable -- the same call, with
the switch off again, gives the oracle's result."""
import ctypes
import os

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2606_26453_b200 import build, workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu

MOE_ERR_TIMEOUT = 8


class Dims(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in "THIEK"]


def test_a_wait_that_runs_out_reports_and_leaves_the_context_usable():
    path = build.build_library(waittest=True)
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    p = ctypes.c_void_p
    lib.moe_grouped_gemm_down.argtypes = [ctypes.POINTER(Dims), p, p, p, p, p]
    lib.moe_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
    lib.moe_test_withhold_first_stage.argtypes = [ctypes.c_int]

    def status():
        out = ctypes.c_int(0)
        assert lib.moe_device_status(ctypes.byref(out)) == 0
        return out.value

    cfg = W.CONFIGS["tiny"]
    host = W.make_workload(cfg)
    ref = O.layer_fwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"])
    h = W.round_to_bf16(ref["H_act"].astype(np.float32))
    h_dev, w_dev = Hh.to_dev_bf16(h), Hh.to_dev_bf16(host["W_down"])
    off = torch.from_numpy(ref["offsets"]).cuda()
    yp = torch.zeros((cfg.R, cfg.H), dtype=torch.bfloat16, device="cuda")
    d = Dims(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K)
    stream = p(torch.cuda.current_stream().cuda_stream)

    def down():
        return lib.moe_grouped_gemm_down(ctypes.byref(d), p(h_dev.data_ptr()), p(w_dev.data_ptr()), p(off.data_ptr()),
                                         p(yp.data_ptr()), stream)

    assert status() == 0
    assert lib.moe_test_withhold_first_stage(1) == 0
    assert down() == 0                                  # the launch itself succeeds
    torch.cuda.synchronize()                            # ... and the kernel returns by itself (bounded waits)
    assert status() == MOE_ERR_TIMEOUT
    assert status() == 0                                # read once, cleared
    assert lib.moe_test_withhold_first_stage(0) == 0
    assert down() == 0
    torch.cuda.synchronize()
    assert status() == 0
    Hh.assert_close(Hh.to_np64(yp), O.down(h, host["W_down"], ref["offsets"]), "Y_perm after a timed-out call",
                    rel_fro=Hh.PER_CALL_FROBENIUS)


@pytest.mark.parametrize("counts", [[60, 70, 0, 62], [700, 513, 64]], ids=["single_cta", "cta_pair"])
def test_block_scaled_kernels_give_up_the_same_way(counts):
    """The same for the two block-scaled FP8 GEMM kernels (more roles wait there: the scale-gather warps, the scale-copy
    warp of the pair kernel): every wait runs out, the status word reads MOE_ERR_TIMEOUT, the next call is correct."""
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    lib = ctypes.CDLL(build.build_library(waittest=True))
    p = ctypes.c_void_p
    lib.moe_grouped_gemm_down_mxfp8.argtypes = [ctypes.POINTER(Dims), p, p, p, p, p, p, p]
    lib.moe_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
    lib.moe_test_withhold_first_stage_mxfp8.argtypes = [ctypes.c_int]

    def status():
        out = ctypes.c_int(0)
        assert lib.moe_device_status(ctypes.byref(out)) == 0
        return out.value

    cfg, host = Hh.ragged_workload(counts, K=1, H=256, I=256, seed=31)
    ref = O.layer_fwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"])
    h = W.round_to_bf16(ref["H_act"].astype(np.float32))
    h_dev, w_dev = Hh.to_dev_bf16(h), Hh.to_dev_bf16(host["W_down"])
    bd = B.dims(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K)
    u8 = lambda n: torch.zeros(n, dtype=torch.uint8, device="cuda")
    hc, hs = u8(cfg.R * cfg.I), u8(B.moe_mxfp8_act_scale_bytes(bd))
    wc, ws = u8(cfg.E * cfg.H * cfg.I), u8(B.moe_mxfp8_w_down_scale_bytes(bd))
    B.moe_mxfp8_quantize_h_act(bd, h_dev, hc, hs)            # operands from the regular library
    B.moe_mxfp8_quantize_w_down(bd, w_dev, wc, ws)
    off = torch.from_numpy(ref["offsets"]).cuda()
    yp = torch.zeros((cfg.R, cfg.H), dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    d = Dims(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K)
    stream = p(torch.cuda.current_stream().cuda_stream)

    def down():
        return lib.moe_grouped_gemm_down_mxfp8(ctypes.byref(d), p(hc.data_ptr()), p(hs.data_ptr()), p(wc.data_ptr()),
                                               p(ws.data_ptr()), p(off.data_ptr()), p(yp.data_ptr()), stream)

    assert status() == 0
    assert lib.moe_test_withhold_first_stage_mxfp8(1) == 0
    assert down() == 0
    torch.cuda.synchronize()                            # the kernel returns by itself
    assert status() == MOE_ERR_TIMEOUT
    assert lib.moe_test_withhold_first_stage_mxfp8(0) == 0
    assert down() == 0
    torch.cuda.synchronize()
    assert status() == 0
    Hh.assert_close(Hh.to_np64(yp), O.down_mxfp8(h, host["W_down"], ref["offsets"]), "Y_perm (MXFP8) after a timed-out call",
                    rel_fro=Hh.PER_CALL_FROBENIUS)
