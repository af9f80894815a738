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
