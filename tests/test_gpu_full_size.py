"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The fp64 oracle cannot evaluate a whole full-size layer in seconds, so it evaluates REDUCED layers
that are exact restrictions of the full one:
  * a token subset (all weights): Y[t], dX[t], dtopk_w[t] of a token depend on that token only;
  * the pairs routed to a few experts, taken as K=1 tokens, with the intermediate dimension
    restricted to a column subset S: dW_gate[e][:,S], dW_up[e][:,S], dW_down[e][S,:] of the full
    layer equal those of the restricted layer, because dY_perm = w*dY does not depend on I.
Indices, offsets and counts are compared in full, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2606_26453_b200 import workloads as W
from tests import helpers as Hh

pytestmark = pytest.mark.gpu

FULL = ["fine_grained", "many_small", "few_large", "imbalanced", "paper_dw1"]


def f32(t):
    return t.to(torch.float32).cpu().numpy()


@pytest.fixture(scope="module", params=FULL)
def full(request):
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    cfg = W.CONFIGS[request.param]
    dev = W.make_workload_device(cfg, torch.device("cuda", 0))
    b = Hh.run_cuda_layer(dev, cfg.E)
    yield cfg, dev, b
    del dev, b
    torch.cuda.empty_cache()


def test_indices_bit_exact(full):
    cfg, dev, b = full
    counts, offsets, r2p, p2r = O.permute_indices(dev["topk_idx"].cpu().numpy(), cfg.E)
    assert np.array_equal(b.counts.cpu().numpy(), counts)
    assert np.array_equal(b.offsets.cpu().numpy(), offsets)
    assert np.array_equal(b.row_to_pair.cpu().numpy(), r2p)
    assert np.array_equal(b.pair_to_row.cpu().numpy(), p2r)
    if cfg.name == "imbalanced":
        assert (counts == 0).sum() == 4          # the configuration's empty experts are really there
    if cfg.name == "paper_dw1":
        assert (counts == 0).sum() >= 3          # the paper's load model leaves several experts without rows
    # packed rows are bit copies of the token rows (sampled rows, checked on the device)
    rows = torch.randint(0, cfg.R, (4096,), device="cuda")
    src = (b.row_to_pair[rows] // cfg.K).long()
    assert torch.equal(b.x_perm[rows], dev["X"][src])


PACKED = [("x_perm", "X_perm"), ("h_act", "H_act"), ("gu", "GU"), ("y_perm", "Y_perm"), ("dy_perm", "dY_perm"),
          ("dh_act", "dH_act"), ("dgu", "dGU"), ("dx_perm", "dX_perm")]


def test_sampled_tokens_against_exact_chain(full):
    """64 tokens (the first and the last among them) through the exact chain with all of their experts' weights:
    Y, dX, dtopk_w of those tokens, and every packed intermediate row that belongs to one of their pairs."""
    cfg, dev, b = full
    rng = np.random.default_rng(cfg.cfg_id)
    toks = np.sort(rng.choice(cfg.T, size=64, replace=False))
    toks[0], toks[-1] = 0, cfg.T - 1
    idx = dev["topk_idx"].cpu().numpy()[toks]
    touched = np.unique(idx)
    remap = -np.ones(cfg.E, dtype=np.int64)
    remap[touched] = np.arange(touched.size)
    tsel = torch.from_numpy(toks).cuda()
    esel = torch.from_numpy(touched).cuda()
    ref = O.layer_fwd_bwd(f32(dev["X"][tsel]), remap[idx].astype(np.int32), dev["topk_w"].cpu().numpy()[toks],
                          f32(dev["W_gate"][esel]), f32(dev["W_up"][esel]), f32(dev["W_down"][esel]),
                          f32(dev["dY"][tsel]))
    Hh.assert_close(Hh.to_np64(b.y[tsel]), ref["Y"], "Y[sample]")
    Hh.assert_close(Hh.to_np64(b.dx[tsel]), ref["dX"], "dX[sample]")
    Hh.assert_close(b.dtopk_w[tsel].cpu().numpy().astype(np.float64), ref["dtopk_w"], "dtopk_w[sample]")
    # row r' of the reduced layer is pair (t', k): the full layer keeps that pair in row pair_to_row[toks[t'] * K + k]
    K = cfg.K
    small_pairs = ref["row_to_pair"].astype(np.int64)
    full_pairs = toks[small_pairs // K] * K + small_pairs % K
    rows = b.pair_to_row[torch.from_numpy(full_pairs).cuda()].long()
    for attr, key in PACKED:
        Hh.assert_close(Hh.to_np64(getattr(b, attr)[rows]), ref[key], key + "[rows of the sampled tokens]")
    # the same tokens through the chain that uses the fused down-dgrad + SwiGLU-backward call
    from paper_2606_26453_b200 import binding as B
    B.layer_backward(b, dev["dY"], dev["topk_w"], dev["W_gate"], dev["W_up"], dev["W_down"], fused_swiglu_bwd=True)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    Hh.assert_close(Hh.to_np64(b.dgu[rows]), ref["dGU"], "fused chain dGU[rows]")
    Hh.assert_close(Hh.to_np64(b.dx_perm[rows]), ref["dX_perm"], "fused chain dX_perm[rows]")
    Hh.assert_close(Hh.to_np64(b.dx[tsel]), ref["dX"], "fused chain dX[sample]")
    B.layer_backward(b, dev["dY"], dev["topk_w"], dev["W_gate"], dev["W_up"], dev["W_down"])   # back to the two-call chain
    torch.cuda.synchronize()


def test_sampled_weight_gradient_blocks_against_exact_chain(full):
    cfg, dev, b = full
    counts = b.counts.cpu().numpy()
    offsets = b.offsets.cpu().numpy()
    nonempty = np.flatnonzero(counts > 0)
    rng = np.random.default_rng(100 + cfg.cfg_id)
    # the largest expert, the smallest one with rows, a random one (an expert without rows is checked for exact zeros)
    chosen = {int(nonempty[np.argmax(counts[nonempty])]), int(nonempty[np.argmin(counts[nonempty])]),
              int(rng.choice(nonempty)), int(nonempty[len(nonempty) // 2])}
    if cfg.name == "few_large":
        chosen = {int(nonempty[0]), int(nonempty[-1])}        # 2k rows x 14336 columns each: two are enough
    chosen = sorted(chosen)
    I = cfg.I
    S = np.concatenate([np.arange(96, 160), np.arange(I - 64, I)])          # straddles a tile edge; last columns
    ssel = torch.from_numpy(S).cuda()
    K = cfg.K
    r2p = b.row_to_pair.cpu().numpy().astype(np.int64)
    pairs = np.concatenate([r2p[offsets[e]:offsets[e + 1]] for e in chosen])
    e_new = np.concatenate([np.full(counts[e], i, dtype=np.int32) for i, e in enumerate(chosen)])
    tok = torch.from_numpy(pairs // K).cuda()
    esel = torch.tensor(chosen, device="cuda")
    w_pairs = dev["topk_w"].reshape(-1)[torch.from_numpy(pairs).cuda()].cpu().numpy()
    ref = O.layer_fwd_bwd(f32(dev["X"][tok]), e_new[:, None], w_pairs[:, None],
                          f32(dev["W_gate"][esel][:, :, ssel]), f32(dev["W_up"][esel][:, :, ssel]),
                          f32(dev["W_down"][esel][:, ssel, :]), f32(dev["dY"][tok]))
    assert np.array_equal(ref["counts"], counts[chosen])
    Hh.assert_close(Hh.to_np64(b.dw_gate[esel][:, :, ssel]), ref["dW_gate"], "dW_gate[block]")
    Hh.assert_close(Hh.to_np64(b.dw_up[esel][:, :, ssel]), ref["dW_up"], "dW_up[block]")
    Hh.assert_close(Hh.to_np64(b.dw_down[esel][:, ssel, :]), ref["dW_down"], "dW_down[block]")
    # the reduced layer's packed intermediates are rows/columns of the full ones too
    rows = torch.from_numpy(np.concatenate([np.arange(offsets[e], offsets[e + 1]) for e in chosen])).cuda()
    Hh.assert_close(Hh.to_np64(b.h_act[rows][:, ssel]), ref["H_act"], "H_act[block]")
    Hh.assert_close(Hh.to_np64(b.dy_perm[rows]), ref["dY_perm"], "dY_perm[rows]")
    Hh.assert_close(Hh.to_np64(b.dh_act[rows][:, ssel]), ref["dH_act"], "dH_act[block]")
    # experts without rows: exact zeros everywhere
    for e in np.flatnonzero(counts == 0):
        assert not bool(b.dw_gate[e].any()) and not bool(b.dw_up[e].any()) and not bool(b.dw_down[e].any())


def test_mxfp8_down_sampled_rows(full):
    """The block-scaled FP8 down projection at full size (the CTA-pair kernel on the four workloads it takes): codes
    and scale bytes of 48 sampled rows bit for bit, and those rows of Y_perm against the exact product of the
    dequantised operands -- the oracle quantises the sampled rows and their experts' weights only.  The row of every
    expert boundary is among the samples.  Run to run the result is the same bits."""
    cfg, dev, b = full
    if cfg.H % 128 or cfg.I % 128:
        pytest.skip("the block-scaled path takes widths that are multiples of 128")
    from paper_2606_26453_b200 import binding as B
    d = b.d
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    hc, hs = u8(cfg.R * cfg.I), u8(B.moe_mxfp8_act_scale_bytes(d))
    wc, ws = u8(cfg.E * cfg.H * cfg.I), u8(B.moe_mxfp8_w_down_scale_bytes(d))
    B.moe_mxfp8_quantize_h_act(d, b.h_act, hc, hs)
    B.moe_mxfp8_quantize_w_down(d, dev["W_down"], wc, ws)
    yq = torch.full((cfg.R, cfg.H), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.moe_grouped_gemm_down_mxfp8(d, hc, hs, wc, ws, b.offsets, yq)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    assert not bool(torch.isnan(yq).any())                       # every row of every expert was written
    offsets = b.offsets.cpu().numpy()
    rng = np.random.default_rng(cfg.cfg_id + 7)
    nonempty = np.flatnonzero(np.diff(offsets) > 0)
    experts = rng.choice(nonempty, size=min(6, nonempty.size), replace=False)
    rows = []
    for e in experts:
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        rows += [lo, hi - 1] + list(rng.integers(lo, hi, size=6))    # first and last row of the expert + 6 inside
    rows = np.array(sorted(set(rows)))
    expert_of = np.searchsorted(offsets, rows, side="right") - 1
    rsel = torch.from_numpy(rows).cuda()
    h_rows = f32(b.h_act[rsel])
    o_codes, o_scales, h_deq = O.mxfp8_quantize(h_rows)
    assert np.array_equal(hc.view(cfg.R, cfg.I)[rsel].cpu().numpy(), o_codes)
    got_scales = hs.view(cfg.I // 128, cfg.R, 4)[:, rsel].cpu().numpy().transpose(1, 0, 2).reshape(rows.size, cfg.I // 32)
    assert np.array_equal(got_scales, o_scales)
    got = Hh.to_np64(yq[rsel])
    want = np.empty_like(got)
    for e in experts:
        wt = np.swapaxes(f32(dev["W_down"][int(e)]), 0, 1)       # [H, I]: contraction last
        w_codes, _, w_deq = O.mxfp8_quantize(wt)
        assert np.array_equal(wc.view(cfg.E, cfg.H, cfg.I)[int(e)].cpu().numpy(), w_codes)
        sel = expert_of == e
        want[sel] = h_deq[sel] @ w_deq.T
    Hh.assert_close(got, want, f"{cfg.name}: Y_perm rows (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    first = yq.clone()
    yq.fill_(float("nan"))
    B.moe_grouped_gemm_down_mxfp8(d, hc, hs, wc, ws, b.offsets, yq)
    torch.cuda.synchronize()
    assert torch.equal(yq, first)


def test_mxfp8_other_gemms_sampled_rows(full):
    """The other three block-scaled FP8 GEMMs at full size -- gate/up forward (with the SwiGLU call), down dgrad,
    gate/up dgrad -- on sampled rows (first and last row of 4 experts + 4 inside each) against the exact products of the
    dequantised operands; the oracle quantises the sampled rows and those experts' weights only."""
    cfg, dev, b = full
    if cfg.H % 128 or cfg.I % 128:
        pytest.skip("the block-scaled path takes widths that are multiples of 128")
    from paper_2606_26453_b200 import binding as B
    d = b.d
    R, E, H, I = cfg.R, cfg.E, cfg.H, cfg.I
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    nan = lambda *shape: torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    offsets = b.offsets.cpu().numpy()
    rng = np.random.default_rng(cfg.cfg_id + 11)
    nonempty = np.flatnonzero(np.diff(offsets) > 0)
    experts = rng.choice(nonempty, size=min(4, nonempty.size), replace=False)
    rows = []
    for e in experts:
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        rows += [lo, hi - 1] + list(rng.integers(lo, hi, size=4))
    rows = np.array(sorted(set(rows)))
    expert_of = np.searchsorted(offsets, rows, side="right") - 1
    rsel = torch.from_numpy(rows).cuda()
    wg = {int(e): f32(dev["W_gate"][int(e)]) for e in experts}
    wu = {int(e): f32(dev["W_up"][int(e)]) for e in experts}
    wd = {int(e): f32(dev["W_down"][int(e)]) for e in experts}

    # gate/up forward: GU rows, then H_act and its codes from the CUDA side's own GU
    xc, xs = u8(R * H), u8(B.moe_mxfp8_x_scale_bytes(d))
    tc, ts = u8(E * 2 * I * H), u8(B.moe_mxfp8_w_gateup_scale_bytes(d))
    gu = nan(R, 2 * I)
    B.moe_mxfp8_quantize_x_perm(d, b.x_perm, xc, xs)
    B.moe_mxfp8_quantize_w_gateup(d, dev["W_gate"], dev["W_up"], tc, ts)
    B.moe_grouped_gemm_gateup_mxfp8(d, xc, xs, tc, ts, b.offsets, gu)
    h, hc, hs = nan(R, I), u8(R * I), u8(B.moe_mxfp8_act_scale_bytes(d))
    B.moe_swiglu_mxfp8(d, gu, h, hc, hs)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0 and not bool(torch.isnan(gu).any()) and not bool(torch.isnan(h).any())
    x_deq = O.mxfp8_quantize(f32(b.x_perm[rsel]))[2]
    want = np.empty((rows.size, 2 * I))
    for e in experts:
        sel = expert_of == e
        g_deq = O.mxfp8_quantize(wg[int(e)].T)[2]                # [I, H]: every gate feature's scales along H
        u_deq = O.mxfp8_quantize(wu[int(e)].T)[2]
        want[sel] = np.concatenate([x_deq[sel] @ g_deq.T, x_deq[sel] @ u_deq.T], axis=1)
    Hh.assert_close(Hh.to_np64(gu[rsel]), want, f"{cfg.name}: GU rows (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    Hh.assert_close(Hh.to_np64(h[rsel]), O.swiglu_fwd(Hh.to_np64(gu[rsel])), f"{cfg.name}: H_act rows from GU",
                    rel_fro=Hh.PER_CALL_FROBENIUS)
    assert np.array_equal(hc.view(R, I)[rsel].cpu().numpy(), O.mxfp8_quantize(Hh.to_np64(h[rsel]))[0])
    del xc, xs, tc, ts, gu, h, hc, hs

    # down dgrad
    dc, ds = u8(R * H), u8(B.moe_mxfp8_dy_scale_bytes(d))
    vc, vs = u8(E * I * H), u8(B.moe_mxfp8_w_down_dgrad_scale_bytes(d))
    dh = nan(R, I)
    B.moe_mxfp8_quantize_dy_perm(d, b.dy_perm, dc, ds)
    B.moe_mxfp8_quantize_w_down_dgrad(d, dev["W_down"], vc, vs)
    B.moe_grouped_gemm_down_dgrad_mxfp8(d, dc, ds, vc, vs, b.offsets, dh)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0 and not bool(torch.isnan(dh).any())
    dy_deq = O.mxfp8_quantize(f32(b.dy_perm[rsel]))[2]
    want = np.empty((rows.size, I))
    for e in experts:
        sel = expert_of == e
        want[sel] = dy_deq[sel] @ O.mxfp8_quantize(wd[int(e)])[2].T     # [I, H] as it lies
    Hh.assert_close(Hh.to_np64(dh[rsel]), want, f"{cfg.name}: dH_act rows (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    del dc, ds, vc, vs, dh

    # gate/up dgrad
    gc, gs = u8(R * 2 * I), u8(B.moe_mxfp8_dgu_scale_bytes(d))
    uc, us = u8(E * H * 2 * I), u8(B.moe_mxfp8_w_gateup_dgrad_scale_bytes(d))
    dx = nan(R, H)
    B.moe_mxfp8_quantize_dgu(d, b.dgu, gc, gs)
    B.moe_mxfp8_quantize_w_gateup_dgrad(d, dev["W_gate"], dev["W_up"], uc, us)
    B.moe_grouped_gemm_gateup_dgrad_mxfp8(d, gc, gs, uc, us, b.offsets, dx)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0 and not bool(torch.isnan(dx).any())
    dgu_deq = O.mxfp8_quantize(f32(b.dgu[rsel]))[2]
    want = np.empty((rows.size, H))
    for e in experts:
        sel = expert_of == e
        want[sel] = dgu_deq[sel, :I] @ O.mxfp8_quantize(wg[int(e)])[2].T + dgu_deq[sel, I:] @ O.mxfp8_quantize(wu[int(e)])[2].T
    Hh.assert_close(Hh.to_np64(dx[rsel]), want, f"{cfg.name}: dX_perm rows (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)


def test_mxfp8_weight_gradients_sampled_experts(full):
    """The block-scaled FP8 weight gradients at full size: the smallest expert with rows, a mid-sized one and every
    expert without rows, on 256 output columns each, against the exact product of the token-quantised operands (the
    oracle quantises those experts' rows only, in blocks of 32 counted from the expert's first row)."""
    cfg, dev, b = full
    if cfg.H % 128 or cfg.I % 128:
        pytest.skip("the block-scaled path takes widths that are multiples of 128")
    from paper_2606_26453_b200 import binding as B
    d = b.d
    R, E, H, I = cfg.R, cfg.E, cfg.H, cfg.I
    u8 = lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
    tok = lambda n: (u8(B.moe_mxfp8_tokens_codes_bytes(d, n)), u8(B.moe_mxfp8_tokens_scale_bytes(d, n)))
    offsets = b.offsets.cpu().numpy()
    counts = np.diff(offsets)
    order = np.argsort(counts, kind="stable")
    nonempty = [int(e) for e in order if counts[e] > 0]
    picks = [nonempty[0], nonempty[len(nonempty) // 2]]
    cols = slice(128, 384)                                   # crosses a 208-column tile boundary

    def expert_ref(a_rows, b_rows, e):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        one = np.array([0, hi - lo])
        return O.wgrad_mxfp8(f32(a_rows[lo:hi]), f32(b_rows[lo:hi]), one)[0]

    (hc, hs), (dc, ds) = tok(I), tok(H)
    B.moe_mxfp8_quantize_tokens(d, b.h_act, I, 0, I, b.offsets, hc, hs)
    B.moe_mxfp8_quantize_tokens(d, b.dy_perm, H, 0, H, b.offsets, dc, ds)
    dwd = torch.full((E, I, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.moe_grouped_gemm_down_wgrad_mxfp8(d, hc, hs, dc, ds, dwd)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0 and not bool(torch.isnan(dwd).any())
    for e in picks:
        want = expert_ref(b.h_act, b.dy_perm[:, cols], e)
        Hh.assert_close(Hh.to_np64(dwd[e][:, cols]), want, f"{cfg.name}: dW_down[{e}] (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    for e in np.flatnonzero(counts == 0):
        assert not bool(dwd[int(e)].any())
    del hc, hs, dc, ds, dwd

    (xc, xs), (gc, gs), (uc, us) = tok(H), tok(I), tok(I)
    B.moe_mxfp8_quantize_tokens(d, b.x_perm, H, 0, H, b.offsets, xc, xs)
    B.moe_mxfp8_quantize_tokens(d, b.dgu, 2 * I, 0, I, b.offsets, gc, gs)
    B.moe_mxfp8_quantize_tokens(d, b.dgu, 2 * I, I, I, b.offsets, uc, us)
    dwg = torch.full((E, H, I), float("nan"), dtype=torch.bfloat16, device="cuda")
    dwu = torch.full((E, H, I), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.moe_grouped_gemm_gateup_wgrad_mxfp8(d, xc, xs, gc, gs, uc, us, dwg, dwu)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0 and not bool(torch.isnan(dwg).any()) and not bool(torch.isnan(dwu).any())
    for e in picks:
        Hh.assert_close(Hh.to_np64(dwg[e][:, cols]), expert_ref(b.x_perm, b.dgu[:, :I][:, cols], e),
                        f"{cfg.name}: dW_gate[{e}] (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
        Hh.assert_close(Hh.to_np64(dwu[e][:, cols]), expert_ref(b.x_perm, b.dgu[:, I:][:, cols], e),
                        f"{cfg.name}: dW_up[{e}] (MXFP8)", rel_fro=Hh.PER_CALL_FROBENIUS)
    for e in np.flatnonzero(counts == 0):
        assert not bool(dwg[int(e)].any()) and not bool(dwu[int(e)].any())


# ------------------------------------------------------------------------------------------------
# every element of every output, where the oracle can afford the whole layer (about 15 s and 45 s of host time)
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["fine_grained", "many_small"])
def test_every_element_against_exact_chain(name):
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    cfg = W.CONFIGS[name]
    dev = W.make_workload_device(cfg, torch.device("cuda", 0))
    b = Hh.run_cuda_layer(dev, cfg.E)
    host = Hh.host_view(dev)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"],
                          host["dY"])
    del host
    for k in ("counts", "offsets", "row_to_pair", "pair_to_row"):
        assert np.array_equal(getattr(b, k).cpu().numpy(), ref[k]), k
    outputs = [("y", "Y"), ("dx", "dX"), ("dw_gate", "dW_gate"), ("dw_up", "dW_up"), ("dw_down", "dW_down")] + PACKED
    for attr, key in outputs:
        Hh.assert_close(getattr(b, attr).to(torch.float32).cpu().numpy(), ref[key], f"{name} {key} (every element)")
    Hh.assert_close(b.dtopk_w.cpu().numpy(), ref["dtopk_w"], f"{name} dtopk_w (every element)")
    # and the chain with the fused down-dgrad + SwiGLU-backward call
    B.layer_backward(b, dev["dY"], dev["topk_w"], dev["W_gate"], dev["W_up"], dev["W_down"], fused_swiglu_bwd=True)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    for attr, key in (("dgu", "dGU"), ("dx_perm", "dX_perm"), ("dx", "dX"), ("dw_gate", "dW_gate"), ("dw_up", "dW_up")):
        Hh.assert_close(getattr(b, attr).to(torch.float32).cpu().numpy(), ref[key], f"{name} fused chain {key} (every element)")
    # run to run the fused call gives the same bits (a race on its shared-memory input blocks would show here)
    first = b.dgu.clone()
    for _ in range(4):
        b.dgu.fill_(float("nan"))
        B.moe_grouped_gemm_down_dgrad_swiglu_bwd(b.d, b.dy_perm, dev["W_down"], b.gu, b.offsets, b.dgu)
        torch.cuda.synchronize()
        assert torch.equal(b.dgu, first)
