"""Seeded random shapes and expert loads through the six block-scaled FP8 GEMMs, against the oracle's exact products of
the dequantised operands.

The fixed cases of test_gpu_mxfp8.py pin the tile edges one knows about (208- and 128-column tiles, 256- and 128-row
tiles, K slices, empty experts); these draw widths (multiples of 128), expert counts and per-expert row counts -- empty
experts, single rows, tile-boundary sizes, one large expert -- on both sides of the single-CTA / CTA-pair threshold.
Operands are the bf16 layer's own intermediates, so every GEMM sees realistic value ranges."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


def draw_case(seed):
    rng = np.random.default_rng(7000 + seed)
    H = 128 * int(rng.integers(1, 5))
    I = 128 * int(rng.integers(1, 5))
    E = int(rng.integers(1, 13))
    K = int(rng.integers(1, min(E, 4) + 1))
    level = [40, 200, 300, 700][seed % 4]                      # around and on both sides of 256 rows per expert
    counts = np.maximum(0, rng.normal(level, 0.4 * level, size=E)).astype(np.int64)
    special = [0, 1, 31, 32, 33, 127, 128, 129, 255, 256, 257, 513]
    for e in rng.choice(E, size=min(E, 3), replace=False):
        counts[e] = special[int(rng.integers(0, len(special)))]
    if E > 2 and seed % 3 == 0:
        counts[int(rng.integers(0, E))] = int(rng.integers(900, 1500))
    if int(counts.sum()) == 0:
        counts[0] = K
    for _ in range(64):
        counts[int(np.argmin(counts))] += (-int(counts.sum())) % K
        T = int(counts.sum()) // K
        if int(counts.max()) <= T:
            break
        counts[int(np.argmax(counts))] = T
    return counts, K, H, I


@pytest.mark.parametrize("seed", list(range(16)))
def test_random_shapes_all_six_fp8_gemms(seed):
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    counts, K, H, I = draw_case(seed)
    if int(counts.sum()) % K or int(counts.max()) > int(counts.sum()) // K:
        pytest.skip("drawn counts cannot be routed without repeating an expert in a token")
    cfg, host = Hh.ragged_workload(list(counts), K=K, H=H, I=I, seed=300 + seed)
    dev = Hh.device_workload(host)
    b = Hh.run_cuda_layer(dev, cfg.E)                          # the bf16 layer: its intermediates are the operands
    d = b.d
    R, E = cfg.R, cfg.E
    offsets = b.offsets.cpu().numpy()
    tag = f"counts={list(counts)} K={K} H={H} I={I}"
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    nan = lambda *shape: torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    close = lambda got, want, what: Hh.assert_close(Hh.to_np64(got), want, f"{what} (MXFP8) {tag}", rel_fro=Hh.PER_CALL_FROBENIUS)
    x_perm, h_act, dy_perm, dgu = (Hh.to_np64(t) for t in (b.x_perm, b.h_act, b.dy_perm, b.dgu))
    wg, wu, wd = host["W_gate"], host["W_up"], host["W_down"]

    # forward: gate/up (+ SwiGLU with its quantiser), down fed by those codes
    xc, xs = u8(R * H), u8(B.moe_mxfp8_x_scale_bytes(d))
    tc, ts = u8(E * 2 * I * H), u8(B.moe_mxfp8_w_gateup_scale_bytes(d))
    gu, h, hc, hs = nan(R, 2 * I), nan(R, I), u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    B.moe_mxfp8_quantize_x_perm(d, b.x_perm, xc, xs)
    B.moe_mxfp8_quantize_w_gateup(d, dev["W_gate"], dev["W_up"], tc, ts)
    B.moe_grouped_gemm_gateup_mxfp8(d, xc, xs, tc, ts, b.offsets, gu)
    B.moe_swiglu_mxfp8(d, gu, h, hc, hs)
    wc, ws = u8(E * H * I), u8(B.moe_mxfp8_w_down_scale_bytes(d))
    yq = nan(R, H)
    B.moe_mxfp8_quantize_w_down(d, dev["W_down"], wc, ws)
    B.moe_grouped_gemm_down_mxfp8(d, hc, hs, wc, ws, b.offsets, yq)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    close(gu, O.gateup_mxfp8(x_perm, wg, wu, offsets), "GU")
    close(h, O.swiglu_fwd(Hh.to_np64(gu)), "H_act from GU")
    assert np.array_equal(hc.view(R, I).cpu().numpy(), O.mxfp8_quantize(Hh.to_np64(h))[0]), tag
    close(yq, O.down_mxfp8(Hh.to_np64(h), wd, offsets), "Y_perm")

    # data gradients
    dc, ds = u8(R * H), u8(B.moe_mxfp8_dy_scale_bytes(d))
    vc, vs = u8(E * I * H), u8(B.moe_mxfp8_w_down_dgrad_scale_bytes(d))
    dh = nan(R, I)
    B.moe_mxfp8_quantize_dy_perm(d, b.dy_perm, dc, ds)
    B.moe_mxfp8_quantize_w_down_dgrad(d, dev["W_down"], vc, vs)
    B.moe_grouped_gemm_down_dgrad_mxfp8(d, dc, ds, vc, vs, b.offsets, dh)
    gc, gs = u8(R * 2 * I), u8(B.moe_mxfp8_dgu_scale_bytes(d))
    uc, us = u8(E * H * 2 * I), u8(B.moe_mxfp8_w_gateup_dgrad_scale_bytes(d))
    dx = nan(R, H)
    B.moe_mxfp8_quantize_dgu(d, b.dgu, gc, gs)
    B.moe_mxfp8_quantize_w_gateup_dgrad(d, dev["W_gate"], dev["W_up"], uc, us)
    B.moe_grouped_gemm_gateup_dgrad_mxfp8(d, gc, gs, uc, us, b.offsets, dx)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    close(dh, O.down_dgrad_mxfp8(dy_perm, wd, offsets), "dH_act")
    close(dx, O.gateup_dgrad_mxfp8(dgu, wg, wu, offsets), "dX_perm")

    # weight gradients
    tok = lambda n: (u8(B.moe_mxfp8_tokens_codes_bytes(d, n)), u8(B.moe_mxfp8_tokens_scale_bytes(d, n)))
    (ac, asc), (bc, bsc), (pc, psc), (qc, qsc), (rc, rsc) = tok(I), tok(H), tok(H), tok(I), tok(I)
    B.moe_mxfp8_quantize_tokens(d, b.h_act, I, 0, I, b.offsets, ac, asc)
    B.moe_mxfp8_quantize_tokens(d, b.dy_perm, H, 0, H, b.offsets, bc, bsc)
    B.moe_mxfp8_quantize_tokens(d, b.x_perm, H, 0, H, b.offsets, pc, psc)
    B.moe_mxfp8_quantize_tokens(d, b.dgu, 2 * I, 0, I, b.offsets, qc, qsc)
    B.moe_mxfp8_quantize_tokens(d, b.dgu, 2 * I, I, I, b.offsets, rc, rsc)
    dwd, dwg, dwu = nan(E, I, H), nan(E, H, I), nan(E, H, I)
    B.moe_grouped_gemm_down_wgrad_mxfp8(d, ac, asc, bc, bsc, dwd)
    B.moe_grouped_gemm_gateup_wgrad_mxfp8(d, pc, psc, qc, qsc, rc, rsc, dwg, dwu)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    close(dwd, O.wgrad_mxfp8(h_act, dy_perm, offsets), "dW_down")
    want = O.wgrad_mxfp8(x_perm, dgu, offsets)
    close(dwg, want[:, :, :I], "dW_gate")
    close(dwu, want[:, :, I:], "dW_up")
    for e in np.flatnonzero(np.diff(offsets) == 0):
        assert not bool(dwd[e].any()) and not bool(dwg[e].any()) and not bool(dwu[e].any()), tag


def test_many_tiny_experts():
    """1024 experts (the largest count the library takes) with 0..5 rows each, and a single expert holding everything:
    the expert tables, the slice prefix and the fixed tile list of the weight gradients at their limits."""
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    rng = np.random.default_rng(99)
    for counts in (list(rng.integers(0, 6, size=1024)), [777]):
        H, I, K = 128, 256, 1
        cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=77)
        dev = Hh.device_workload(host)
        b = Hh.run_cuda_layer(dev, cfg.E)
        d = b.d
        R, E = cfg.R, cfg.E
        offsets = b.offsets.cpu().numpy()
        u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
        nan = lambda *shape: torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        hc, hs = u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
        wc, ws = u8(E * H * I), u8(B.moe_mxfp8_w_down_scale_bytes(d))
        yq = nan(R, H)
        B.moe_mxfp8_quantize_h_act(d, b.h_act, hc, hs)
        B.moe_mxfp8_quantize_w_down(d, dev["W_down"], wc, ws)
        B.moe_grouped_gemm_down_mxfp8(d, hc, hs, wc, ws, b.offsets, yq)
        tok = lambda n: (u8(B.moe_mxfp8_tokens_codes_bytes(d, n)), u8(B.moe_mxfp8_tokens_scale_bytes(d, n)))
        (ac, asc), (bc, bsc) = tok(I), tok(H)
        B.moe_mxfp8_quantize_tokens(d, b.h_act, I, 0, I, b.offsets, ac, asc)
        B.moe_mxfp8_quantize_tokens(d, b.dy_perm, H, 0, H, b.offsets, bc, bsc)
        dwd = nan(E, I, H)
        B.moe_grouped_gemm_down_wgrad_mxfp8(d, ac, asc, bc, bsc, dwd)
        torch.cuda.synchronize()
        assert B.moe_device_status() == 0
        Hh.assert_close(Hh.to_np64(yq), O.down_mxfp8(Hh.to_np64(b.h_act), host["W_down"], offsets), f"Y_perm (MXFP8), E={E}",
                        rel_fro=Hh.PER_CALL_FROBENIUS)
        Hh.assert_close(Hh.to_np64(dwd), O.wgrad_mxfp8(Hh.to_np64(b.h_act), Hh.to_np64(b.dy_perm), offsets),
                        f"dW_down (MXFP8), E={E}", rel_fro=Hh.PER_CALL_FROBENIUS)
        for e in np.flatnonzero(np.diff(offsets) == 0):
            assert not bool(dwd[e].any())
