"""Block-scaled FP8 (MXFP8) calls through the C ABI against the oracle's quantiser and quantised products.

Code and scale buffers start out as 0xFF bytes: as a scale that is NaN, so a kernel that consumed a byte its quantiser
never wrote would poison its output.

Integer results (element codes, scale bytes) are compared bit for bit: both sides decide them on exact values.  The GEMM
is held to the per-call bound of the bf16 kernels against the EXACT product of the dequantised operands (products of
two E4M3 values and their power-of-two scales are exact in fp32; what remains is fp32 accumulation and the one rounding
of the output to bf16).  Against the unquantised layer the result is a few per cent off by construction: stated, not
tested against the bf16 tolerances."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2606_26453_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2606_26453_b200 import binding
    binding.load_library()
    return binding


def _act_scales_from_layout(raw, R, I):
    """[I/128][R][4] bytes -> [R, I/32]"""
    return raw.reshape(I // 128, R, 4).transpose(1, 0, 2).reshape(R, I // 32)


def _w_scales_from_layout(raw, E, H, I):
    """[E][H/128][I/128][512] bytes with byte (h%32)*16 + ((h%128)/32)*4 + b%4 -> [E, H, I/32]"""
    g = raw.reshape(E, H // 128, I // 128, 32, 4, 4)          # [..., h%32, (h%128)/32, b%4]
    return g.transpose(0, 1, 4, 3, 2, 5).reshape(E, H, I // 32)


def _w_scales_pair_layout(scales, E, H, I):   # H = output features, I = contraction of the GEMM in question
    """[E, H, I/32] -> the second copy of the weight scales, in the tiling of the CTA-pair kernel:
    [E][ceil(H/208)][I/128][2 blocks][h' % 32][(h' % 128) / 32][b % 4] with h' = h % 208; also the mask of written bytes"""
    n_tiles = (H + 207) // 208
    out = np.zeros((E, n_tiles, I // 128, 2, 32, 4, 4), dtype=np.uint8)
    written = np.zeros(out.shape, dtype=bool)
    h = np.arange(H)
    c = h % 208
    for b in range(I // 32):
        out[:, h // 208, b // 4, c >> 7, c % 32, (c % 128) // 32, b % 4] = scales[:, :, b]
        written[:, h // 208, b // 4, c >> 7, c % 32, (c % 128) // 32, b % 4] = True
    return out.reshape(-1), written.reshape(-1)


CASES = {
    "one_tile": ([128], 1, 128, 128),
    "ragged": ([0, 1, 127, 0, 129, 128, 300, 15, 0], 2, 256, 384),
    "wide": ([200, 0, 31, 290, 1], 2, 384, 1408),              # 11 slices of the contraction, 3 column tiles
    "many_tiles": ([700, 513, 64], 1, 128, 256),                # >= 256 rows per expert on average: CTA pairs from here on
    "pair_narrow_edge": ([300, 256, 511, 1], 2, 256, 256),      # column tiles of 208 and 48
    "pair_wide": ([700, 0, 514, 300, 1000], 2, 640, 384),       # column tiles 208, 208, 208, 16; an empty expert
    "pair_one_row_tiles": ([257, 1, 769], 1, 384, 128),         # second CTA's rows empty / one row into the next tile
}


@pytest.mark.parametrize("name", list(CASES))
def test_quantisers_and_gemm_against_the_oracle(B, name):
    counts, K, H, I = CASES[name]
    cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=21)
    ref = O.layer_fwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"])
    R, E = cfg.R, cfg.E
    d = B.dims(cfg.T, H, I, E, K)
    # the activation as the CUDA side sees it: the oracle's H_act rounded to bf16, with a few awkward values put in
    h = W.round_to_bf16(ref["H_act"].astype(np.float32))
    h[0, :32] = 0.0                                  # an all-zero block
    h[min(3, R - 1), 32:64] = 2.0 ** -100            # tiny block
    h[R - 1, I - 32:] = np.linspace(-500.0, 500.0, 32, dtype=np.float32)   # includes values that saturate after scaling
    h = W.round_to_bf16(h)
    w = host["W_down"].copy()
    w[0, :32, 0] = 0.0
    h_dev, w_dev = Hh.to_dev_bf16(h), Hh.to_dev_bf16(w)
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    hc, hs = u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    wc, ws = u8(E * H * I), u8(B.moe_mxfp8_w_down_scale_bytes(d))
    n_single = E * (H // 128) * (I // 128) * 512
    assert hs.numel() == (I // 128) * R * 4 and ws.numel() == n_single + E * ((H + 207) // 208) * (I // 128) * 1024
    B.moe_mxfp8_quantize_h_act(d, h_dev, hc, hs)
    B.moe_mxfp8_quantize_w_down(d, w_dev, wc, ws)
    torch.cuda.synchronize()
    o_hc, o_hs, h_deq = O.mxfp8_quantize(h)
    wt = np.swapaxes(w, 1, 2)                        # [E, H, I]
    o_wc, o_ws, _ = O.mxfp8_quantize(wt)
    assert np.array_equal(_act_scales_from_layout(hs.cpu().numpy(), R, I), o_hs)
    assert np.array_equal(hc.cpu().numpy().reshape(R, I), o_hc)
    ws_host = ws.cpu().numpy()
    assert np.array_equal(_w_scales_from_layout(ws_host[:n_single], E, H, I), o_ws)
    want_pair, written = _w_scales_pair_layout(o_ws, E, H, I)
    assert np.array_equal(ws_host[n_single:][written], want_pair[written])
    assert np.all(ws_host[n_single:][~written] == 0xFF)          # bytes no column owns are left alone
    assert np.array_equal(wc.cpu().numpy().reshape(E, H, I), o_wc)
    # the GEMM on the quantised operands
    yp = torch.full((R, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    off = torch.from_numpy(ref["offsets"]).cuda()
    B.moe_grouped_gemm_down_mxfp8(d, hc, hs, wc, ws, off, yp)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    o_y = O.down_mxfp8(h, w, ref["offsets"])
    Hh.assert_close(Hh.to_np64(yp), o_y, f"{name}: Y_perm (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    # for orientation: distance to the unquantised product (a few per cent: the format, not the kernel)
    exact = O.down(h, w, ref["offsets"])
    rel = np.linalg.norm(Hh.to_np64(yp) - exact) / np.linalg.norm(exact)
    assert rel < 0.08


def _w_scales_single_layout(scales, E, N, K):
    """[E, N, K/32] -> [E][N/128][K/128][n % 32][(n % 128) / 32][b % 4] (the first copy of the weight scales)"""
    g = scales.reshape(E, N // 128, 4, 32, K // 128, 4)          # [e, n/128, (n%128)/32, n%32, b/4, b%4]
    return g.transpose(0, 1, 4, 3, 2, 5).reshape(-1)


@pytest.mark.parametrize("name", list(CASES))
def test_down_dgrad_quantisers_and_gemm_against_the_oracle(B, name):
    """dH_act = Q(dY_perm) . Q(W_down[e])^T with both operands quantised along H, on the same two GEMM kernels."""
    counts, K, H, I = CASES[name]
    cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=23)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"],
                          host["dY"])
    R, E = cfg.R, cfg.E
    d = B.dims(cfg.T, H, I, E, K)
    dy = W.round_to_bf16(ref["dY_perm"].astype(np.float32))
    dy[0, :32] = 0.0
    dy[R - 1, H - 32:] = np.linspace(-3000.0, 3000.0, 32, dtype=np.float32)
    dy = W.round_to_bf16(dy)
    w = host["W_down"].copy()
    w[0, 0, :32] = 0.0
    dy_dev, w_dev = Hh.to_dev_bf16(dy), Hh.to_dev_bf16(w)
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    dc, ds = u8(R * H), u8(B.moe_mxfp8_dy_scale_bytes(d))
    wc, ws = u8(E * I * H), u8(B.moe_mxfp8_w_down_dgrad_scale_bytes(d))
    n_single = E * (I // 128) * (H // 128) * 512
    assert ds.numel() == (H // 128) * R * 4 and ws.numel() == n_single + E * ((I + 207) // 208) * (H // 128) * 1024
    B.moe_mxfp8_quantize_dy_perm(d, dy_dev, dc, ds)
    B.moe_mxfp8_quantize_w_down_dgrad(d, w_dev, wc, ws)
    torch.cuda.synchronize()
    o_dc, o_ds, _ = O.mxfp8_quantize(dy)
    o_wc, o_ws, _ = O.mxfp8_quantize(w)              # [E, I, H]: along H as it lies
    assert np.array_equal(_act_scales_from_layout(ds.cpu().numpy(), R, H), o_ds)
    assert np.array_equal(dc.cpu().numpy().reshape(R, H), o_dc)
    assert np.array_equal(wc.cpu().numpy().reshape(E, I, H), o_wc)
    ws_host = ws.cpu().numpy()
    assert np.array_equal(ws_host[:n_single], _w_scales_single_layout(o_ws, E, I, H))
    want_pair, written = _w_scales_pair_layout(o_ws, E, I, H)
    assert np.array_equal(ws_host[n_single:][written], want_pair[written])
    assert np.all(ws_host[n_single:][~written] == 0xFF)
    dh = torch.full((R, I), float("nan"), dtype=torch.bfloat16, device="cuda")
    off = torch.from_numpy(ref["offsets"]).cuda()
    B.moe_grouped_gemm_down_dgrad_mxfp8(d, dc, ds, wc, ws, off, dh)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    Hh.assert_close(Hh.to_np64(dh), O.down_dgrad_mxfp8(dy, w, ref["offsets"]), f"{name}: dH_act (MXFP8)",
                    rel_fro=Hh.PER_CALL_FROBENIUS)
    exact = O.down_bwd(dy, np.zeros((R, I)), w, ref["offsets"])[0]
    assert np.linalg.norm(Hh.to_np64(dh) - exact) / np.linalg.norm(exact) < 0.08


@pytest.mark.parametrize("name", list(CASES))
def test_gateup_dgrad_quantisers_and_gemm_against_the_oracle(B, name):
    """dX_perm = Q(dGU) . Q([W_gate[e] | W_up[e]])^T, contraction over the 2I gate and up features."""
    counts, K, H, I = CASES[name]
    cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=25)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"],
                          host["dY"])
    R, E = cfg.R, cfg.E
    d = B.dims(cfg.T, H, I, E, K)
    dgu = W.round_to_bf16(ref["dGU"].astype(np.float32))
    dgu[0, I - 32:I + 32] = 0.0                      # all-zero blocks on both sides of the gate/up boundary
    dgu[R - 1, :32] = np.linspace(-9.0, 9.0, 32, dtype=np.float32)
    dgu = W.round_to_bf16(dgu)
    wg, wu = host["W_gate"].copy(), host["W_up"].copy() * 3.0
    wu = W.round_to_bf16(wu)
    dgu_dev, wg_dev, wu_dev = Hh.to_dev_bf16(dgu), Hh.to_dev_bf16(wg), Hh.to_dev_bf16(wu)
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    gc, gs = u8(R * 2 * I), u8(B.moe_mxfp8_dgu_scale_bytes(d))
    wc, ws = u8(E * H * 2 * I), u8(B.moe_mxfp8_w_gateup_dgrad_scale_bytes(d))
    n_single = E * (H // 128) * (2 * I // 128) * 512
    assert gs.numel() == (2 * I // 128) * R * 4 and ws.numel() == n_single + E * ((H + 207) // 208) * (2 * I // 128) * 1024
    B.moe_mxfp8_quantize_dgu(d, dgu_dev, gc, gs)
    B.moe_mxfp8_quantize_w_gateup_dgrad(d, wg_dev, wu_dev, wc, ws)
    torch.cuda.synchronize()
    o_gc, o_gs, _ = O.mxfp8_quantize(dgu)
    o_wc, o_ws, _ = O.mxfp8_quantize(np.concatenate([wg, wu], axis=2))     # [E, H, 2I]: blocks never straddle I
    assert np.array_equal(_act_scales_from_layout(gs.cpu().numpy(), R, 2 * I), o_gs)
    assert np.array_equal(gc.cpu().numpy().reshape(R, 2 * I), o_gc)
    assert np.array_equal(wc.cpu().numpy().reshape(E, H, 2 * I), o_wc)
    ws_host = ws.cpu().numpy()
    assert np.array_equal(ws_host[:n_single], _w_scales_single_layout(o_ws, E, H, 2 * I))
    want_pair, written = _w_scales_pair_layout(o_ws, E, H, 2 * I)
    assert np.array_equal(ws_host[n_single:][written], want_pair[written])
    assert np.all(ws_host[n_single:][~written] == 0xFF)
    dx = torch.full((R, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    off = torch.from_numpy(ref["offsets"]).cuda()
    B.moe_grouped_gemm_gateup_dgrad_mxfp8(d, gc, gs, wc, ws, off, dx)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    Hh.assert_close(Hh.to_np64(dx), O.gateup_dgrad_mxfp8(dgu, wg, wu, ref["offsets"]), f"{name}: dX_perm (MXFP8)",
                    rel_fro=Hh.PER_CALL_FROBENIUS)
    exact = O.gateup_bwd_from_dgu(dgu, np.zeros((R, H)), wg, wu, ref["offsets"])[0]
    assert np.linalg.norm(Hh.to_np64(dx) - exact) / np.linalg.norm(exact) < 0.08


@pytest.mark.parametrize("name", list(CASES))
def test_gateup_forward_and_fused_swiglu_quantiser_against_the_oracle(B, name):
    """GU = [Q(X_perm) . Q(W_gate[e]) | Q(X_perm) . Q(W_up[e])] (contraction over H), then H_act = silu(g) * u with its
    block-scaled FP8 form from the same call, then the FP8 down projection fed by those codes: the forward chain."""
    counts, K, H, I = CASES[name]
    cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=27)
    ref = O.layer_fwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"])
    R, E = cfg.R, cfg.E
    d = B.dims(cfg.T, H, I, E, K)
    x = W.round_to_bf16(ref["X_perm"].astype(np.float32))
    x[0, :32] = 0.0
    wg, wu = host["W_gate"].copy(), W.round_to_bf16(host["W_up"] * 2.0)
    wg[0, :32, 0] = 0.0
    x_dev, wg_dev, wu_dev = Hh.to_dev_bf16(x), Hh.to_dev_bf16(wg), Hh.to_dev_bf16(wu)
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    xc, xs = u8(R * H), u8(B.moe_mxfp8_x_scale_bytes(d))
    wc, ws = u8(E * 2 * I * H), u8(B.moe_mxfp8_w_gateup_scale_bytes(d))
    n_single = E * (2 * I // 128) * (H // 128) * 512
    assert xs.numel() == (H // 128) * R * 4 and ws.numel() == n_single + E * ((2 * I + 207) // 208) * (H // 128) * 1024
    B.moe_mxfp8_quantize_x_perm(d, x_dev, xc, xs)
    B.moe_mxfp8_quantize_w_gateup(d, wg_dev, wu_dev, wc, ws)
    torch.cuda.synchronize()
    o_xc, o_xs, _ = O.mxfp8_quantize(x)
    wt = np.concatenate([np.swapaxes(wg, 1, 2), np.swapaxes(wu, 1, 2)], axis=1)      # [E, 2I, H]: contraction last
    o_wc, o_ws, _ = O.mxfp8_quantize(wt)
    assert np.array_equal(_act_scales_from_layout(xs.cpu().numpy(), R, H), o_xs)
    assert np.array_equal(xc.cpu().numpy().reshape(R, H), o_xc)
    assert np.array_equal(wc.cpu().numpy().reshape(E, 2 * I, H), o_wc)
    ws_host = ws.cpu().numpy()
    assert np.array_equal(ws_host[:n_single], _w_scales_single_layout(o_ws, E, 2 * I, H))
    want_pair, written = _w_scales_pair_layout(o_ws, E, 2 * I, H)
    assert np.array_equal(ws_host[n_single:][written], want_pair[written])
    assert np.all(ws_host[n_single:][~written] == 0xFF)
    gu = torch.full((R, 2 * I), float("nan"), dtype=torch.bfloat16, device="cuda")
    off = torch.from_numpy(ref["offsets"]).cuda()
    B.moe_grouped_gemm_gateup_mxfp8(d, xc, xs, wc, ws, off, gu)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    Hh.assert_close(Hh.to_np64(gu), O.gateup_mxfp8(x, wg, wu, ref["offsets"]), f"{name}: GU (MXFP8)",
                    rel_fro=Hh.PER_CALL_FROBENIUS)
    # the activation of the CUDA side's own GU, and the quantised form of the CUDA side's own H_act (decided on exact values)
    h = torch.full((R, I), float("nan"), dtype=torch.bfloat16, device="cuda")
    hc, hs = u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    B.moe_swiglu_mxfp8(d, gu, h, hc, hs)
    torch.cuda.synchronize()
    Hh.assert_close(Hh.to_np64(h), O.swiglu_fwd(Hh.to_np64(gu)), f"{name}: H_act from GU", rel_fro=Hh.PER_CALL_FROBENIUS)
    o_hc, o_hs, _ = O.mxfp8_quantize(Hh.to_np64(h))
    assert np.array_equal(hc.cpu().numpy().reshape(R, I), o_hc)
    assert np.array_equal(_act_scales_from_layout(hs.cpu().numpy(), R, I), o_hs)
    # ... which equals what the stand-alone activation quantiser makes of the same H_act
    hc2, hs2 = u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    B.moe_mxfp8_quantize_h_act(d, h, hc2, hs2)
    torch.cuda.synchronize()
    assert torch.equal(hc, hc2) and torch.equal(hs, hs2)


def _oracle_tokens_layout(x, offsets):
    """What moe_mxfp8_quantize_tokens must produce for x [R, n]: (codes_t [n, n_slices*128], scale bytes
    [n_slices, n, 4], slice_prefix) -- every column quantised by the oracle in expert-aligned blocks of 32 rows."""
    E = len(offsets) - 1
    n = x.shape[1]
    sp = np.concatenate([[0], np.cumsum([(offsets[e + 1] - offsets[e] + 127) // 128 for e in range(E)])]).astype(np.int64)
    codes = np.zeros((n, int(sp[-1]) * 128), dtype=np.uint8)
    scales = np.zeros((int(sp[-1]), n, 4), dtype=np.uint8)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        width = int(sp[e + 1] - sp[e]) * 128
        xt = np.zeros((n, width))
        xt[:, :hi - lo] = x[lo:hi].T
        c, sc, _ = O.mxfp8_quantize(xt)                      # along the padded token axis
        codes[:, sp[e] * 128: sp[e] * 128 + width] = c
        scales[sp[e]:sp[e + 1]] = sc.reshape(n, -1, 4).transpose(1, 0, 2)
    return codes, scales, sp


WGRAD_CASES = {
    "one_slice": ([100], 1, 128, 128),
    "ragged": ([0, 1, 127, 0, 129, 128, 300, 15, 0], 2, 256, 384),          # empty experts, short last blocks
    "wide": ([200, 0, 31, 290, 1], 2, 384, 1408),                            # M and N tiles with remainders
    "big_expert": ([1500, 513, 64], 1, 256, 256),                            # many K slices per tile
}


@pytest.mark.parametrize("name", list(WGRAD_CASES))
def test_weight_gradients_token_quantiser_and_gemm_against_the_oracle(B, name):
    """dW_down = Q(H_act)^T Q(dY_perm) and [dW_gate | dW_up] = Q(X_perm)^T Q(dGU) per expert, operands quantised along
    the token axis in expert-aligned blocks of 32 rows."""
    counts, K, H, I = WGRAD_CASES[name]
    cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=29)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"],
                          host["dY"])
    R, E = cfg.R, cfg.E
    offsets = ref["offsets"]
    d = B.dims(cfg.T, H, I, E, K)
    bf = lambda a: W.round_to_bf16(np.asarray(a, dtype=np.float32))
    x, h, dy, dgu = bf(ref["X_perm"]), bf(ref["H_act"]), bf(ref["dY_perm"]), bf(ref["dGU"])
    x[0, :] = 0.0                                              # a column block that starts with a zero row
    off = torch.from_numpy(offsets).cuda()
    P = ((R + 127) // 128) * 128 + 128 * E
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")

    def quantise(t_host, col0, n):
        t_dev = Hh.to_dev_bf16(t_host)
        codes, scales = u8(B.moe_mxfp8_tokens_codes_bytes(d, n)), u8(B.moe_mxfp8_tokens_scale_bytes(d, n))
        assert codes.numel() == n * P
        B.moe_mxfp8_quantize_tokens(d, t_dev, t_host.shape[1], col0, n, off, codes, scales)
        torch.cuda.synchronize()
        o_codes, o_scales, sp = _oracle_tokens_layout(t_host[:, col0:col0 + n], offsets)
        n_sl = int(sp[-1])
        assert np.array_equal(scales[:4 * (E + 1)].cpu().numpy().view(np.int32), sp.astype(np.int32))
        assert np.array_equal(codes.view(n, P)[:, :n_sl * 128].cpu().numpy(), o_codes)
        words = scales[8192: 8192 + (P // 128) * n * 4].view(P // 128, n, 4)[:n_sl].cpu().numpy()
        assert np.array_equal(words, o_scales)
        # the same bytes in the pair tiling
        atoms = scales[8192 + (P // 128) * n * 4:].view((n + 207) // 208, P // 128, 2, 32, 4, 4).cpu().numpy()
        f = np.arange(n)
        c = f % 208
        got = atoms[f // 208, :n_sl, c >> 7, c % 32, (c % 128) // 32, :]          # [n, n_sl, 4]
        assert np.array_equal(got.transpose(1, 0, 2), o_scales)
        return codes, scales

    hc, hs = quantise(h, 0, I)
    dc, ds = quantise(dy, 0, H)
    dwd = torch.full((E, I, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.moe_grouped_gemm_down_wgrad_mxfp8(d, hc, hs, dc, ds, dwd)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    want = O.wgrad_mxfp8(h, dy, offsets)
    Hh.assert_close(Hh.to_np64(dwd), want, f"{name}: dW_down (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    for e in np.flatnonzero(np.diff(offsets) == 0):
        assert not bool(dwd[e].any())                          # exact zeros for an expert without rows

    xc, xs = quantise(x, 0, H)
    gc, gs = quantise(dgu, 0, I)
    uc, us = quantise(dgu, I, I)
    dwg = torch.full((E, H, I), float("nan"), dtype=torch.bfloat16, device="cuda")
    dwu = torch.full((E, H, I), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.moe_grouped_gemm_gateup_wgrad_mxfp8(d, xc, xs, gc, gs, uc, us, dwg, dwu)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    want = O.wgrad_mxfp8(x, dgu, offsets)                      # [E, H, 2I]
    Hh.assert_close(Hh.to_np64(dwg), want[:, :, :I], f"{name}: dW_gate (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    Hh.assert_close(Hh.to_np64(dwu), want[:, :, I:], f"{name}: dW_up (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    exact = O.gateup_bwd_from_dgu(dgu, x, host["W_gate"], host["W_up"], offsets)[1]
    assert np.linalg.norm(Hh.to_np64(dwg) - exact) / np.linalg.norm(exact) < 0.08


@pytest.mark.parametrize("name", ["ragged", "wide", "pair_wide"])
def test_swiglu_backward_with_fused_quantiser_equals_the_two_calls(B, name):
    """moe_swiglu_bwd_mxfp8 = moe_swiglu_bwd followed by moe_mxfp8_quantize_dgu, bit for bit (dGU, codes, scales); dGU is
    also held to the oracle's SwiGLU backward like the unfused call."""
    counts, K, H, I = CASES[name]
    cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=33)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"],
                          host["dY"])
    R = cfg.R
    d = B.dims(cfg.T, H, I, cfg.E, K)
    dh = Hh.to_dev_bf16(W.round_to_bf16(ref["dH_act"].astype(np.float32)))
    gu = Hh.to_dev_bf16(W.round_to_bf16(ref["GU"].astype(np.float32)))
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    nan = lambda *shape: torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    dgu1, c1, s1 = nan(R, 2 * I), u8(R * 2 * I), u8(B.moe_mxfp8_dgu_scale_bytes(d))
    B.moe_swiglu_bwd(d, dh, gu, dgu1)
    B.moe_mxfp8_quantize_dgu(d, dgu1, c1, s1)
    dgu2, c2, s2 = nan(R, 2 * I), u8(R * 2 * I), u8(B.moe_mxfp8_dgu_scale_bytes(d))
    B.moe_swiglu_bwd_mxfp8(d, dh, gu, dgu2, c2, s2)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    assert torch.equal(dgu1, dgu2) and torch.equal(c1, c2) and torch.equal(s1, s2)
    Hh.assert_close(Hh.to_np64(dgu2), O.swiglu_bwd(Hh.to_np64(dh), Hh.to_np64(gu)), f"{name}: dGU", rel_fro=Hh.PER_CALL_FROBENIUS)


def test_shapes_the_block_scaled_path_does_not_take_are_refused(B):
    d = B.dims(64, 192, 128, 2, 1)                   # H not a multiple of 128
    assert B.moe_mxfp8_act_scale_bytes(d) == 0
    t = torch.zeros(64 * 192, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.MoeError) as ei:
        B.moe_mxfp8_quantize_h_act(d, t, t, t)
    assert ei.value.status == 3
