"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded
inputs.  Indices, offsets and counts bit-exact; floating-point outputs and gradients within
max|err| <= 2e-2 * max|ref| and relative Frobenius error <= 5e-3.

Per-call tests feed each entry point inputs taken from the ORACLE's chain (rounded to bf16), so a
failure names one kernel; end-to-end tests run the whole CUDA chain against the unrounded oracle."""
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


# a small configuration whose expert sizes hit every tile edge: empty experts first, last and adjacent,
# single-row, 127/128/129 rows, more than two row tiles; I is not a multiple of 256.
RAGGED_COUNTS = [0, 1, 127, 0, 0, 129, 128, 300, 15, 0]
CASES = {
    "tiny": lambda: (W.CONFIGS["tiny"], W.make_workload(W.CONFIGS["tiny"])),
    "ragged": lambda: Hh.ragged_workload(RAGGED_COUNTS, K=2, H=256, I=384, seed=1),
    "ragged_k5": lambda: Hh.ragged_workload([65, 0, 250, 33, 17, 640], K=5, H=384, I=128, seed=2),
    # H and I multiples of 64 only (the paper's 2880 = 45 * 64): partial column tiles everywhere
    "ragged_64": lambda: Hh.ragged_workload([200, 0, 31, 290, 1], K=2, H=192, I=320, seed=4),
    "pair_64": lambda: Hh.ragged_workload([600, 540, 0, 700], K=2, H=320, I=192, seed=6),
    # CTA-pair kernels whose last 256-row tile per expert holds 100, exactly 128, 65 and 129 rows (the second CTA's
    # half of the tile partly or wholly past the expert's end), plus one expert of several full tiles
    "pair_half": lambda: Hh.ragged_workload([356, 640, 321, 900, 385], K=2, H=256, I=320, seed=8),
}


@pytest.fixture(scope="module", params=list(CASES))
def case(request):
    cfg, host = CASES[request.param]()
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"],
                          host["W_down"], host["dY"])
    return cfg, host, ref


def _i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def _bf(a):
    return Hh.to_dev_bf16(W.round_to_bf16(np.asarray(a, dtype=np.float32)))


def _r(a):
    """What the CUDA side sees after the upload: the oracle value rounded to bf16."""
    return W.round_to_bf16(np.asarray(a, dtype=np.float32))


# ------------------------------------------------------------------------------------------------
# a1: permutation, bit-exact
# ------------------------------------------------------------------------------------------------
def _check_permute(B, idx_np, E, X_np=None):
    T, K = idx_np.shape
    H = 128 if X_np is None else X_np.shape[1]
    d = B.dims(T, H, 128, E, K)
    R = T * K
    idx = _i32(idx_np)
    counts = torch.full((E,), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((E + 1,), -7, dtype=torch.int32, device="cuda")
    r2p = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    p2r = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(B.moe_permute_workspace_bytes(d), 16), dtype=torch.uint8, device="cuda")
    x = xp = None
    if X_np is not None:
        x = Hh.to_dev_bf16(X_np)
        xp = torch.full((R, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.moe_permute(d, x, idx, xp, counts, offsets, r2p, p2r, ws)
    torch.cuda.synchronize()
    oc, oo, or2p, op2r = O.permute_indices(idx_np, E)
    assert np.array_equal(counts.cpu().numpy(), oc)
    assert np.array_equal(offsets.cpu().numpy(), oo)
    assert np.array_equal(r2p.cpu().numpy(), or2p)
    assert np.array_equal(p2r.cpu().numpy(), op2r)
    if X_np is not None:
        ref = O.permute(X_np, idx_np, E)[0]
        assert np.array_equal(Hh.to_np64(xp), ref)          # a bit copy of bf16 rows


@pytest.mark.parametrize("T,E,K,seed", [(1, 1, 1, 0), (5, 3, 2, 1), (256, 8, 2, 2), (1000, 64, 6, 3), (4099, 128, 8, 4),
                                        (300, 1024, 3, 5), (777, 5, 5, 6),
                                        (4096, 256, 8, 7), (4097, 256, 8, 8), (1000, 257, 8, 9)])   # 16+ block-chunks
def test_permute_indices_random_with_duplicates(B, T, E, K, seed):
    rng = np.random.default_rng(seed)
    idx = rng.integers(0, E, size=(T, K)).astype(np.int32)
    if E > 3:
        idx[idx == 2] = 0
    _check_permute(B, idx, E)


def test_permute_rows_and_indices(B, case):
    cfg, host, ref = case
    _check_permute(B, host["topk_idx"], cfg.E, host["X"])


@pytest.mark.parametrize("T,H,E,K,seed", [(3, 64, 4, 2, 0),            # fewer tokens than one block takes
                                          (37, 8256, 40, 32, 1),       # rows longer than one bulk-copy segment, K = 32
                                          (1027, 8192, 9, 3, 2),       # 16 KB rows, a ragged last block
                                          (6001, 192, 130, 7, 3)])     # several histogram chunks, odd K
def test_permute_rows_odd_shapes(B, T, H, E, K, seed):
    rng = np.random.default_rng(seed)
    idx = np.stack([rng.permutation(E)[:K] for _ in range(T)]).astype(np.int32)
    X = W.round_to_bf16(rng.standard_normal((T, H), dtype=np.float32))
    _check_permute(B, idx, E, X)


def test_permute_drops_invalid_expert_ids_and_reports_them(B):
    """Expert ids outside [0, E) are a precondition violation: the pairs are dropped (no row, no fault, nothing
    written outside the outputs) and MOE_ERR_BAD_INDEX lands in the device status word; the valid pairs are
    ranked as the stable sort of the valid pairs alone."""
    T, H, E, K = 700, 128, 12, 4
    rng = np.random.default_rng(11)
    idx_np = rng.integers(0, E, size=(T, K)).astype(np.int32)
    flat = idx_np.reshape(-1)
    bad_at = rng.choice(flat.size, size=25, replace=False)
    flat[bad_at] = rng.choice(np.array([-1, -7, E, E + 1, 2 ** 30, -2 ** 31], dtype=np.int64), size=25).astype(np.int32)
    flat[0] = E                      # the very first and the very last pair too
    flat[-1] = -1
    valid = (flat >= 0) & (flat < E)
    R, n_valid = flat.size, int(valid.sum())
    X = W.round_to_bf16(rng.standard_normal((T, H), dtype=np.float32))
    d = B.dims(T, H, 128, E, K)
    guard = 64
    counts = torch.full((E + 2 * guard,), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((E + 1 + 2 * guard,), -7, dtype=torch.int32, device="cuda")
    r2p = torch.full((R + 2 * guard,), -7, dtype=torch.int32, device="cuda")
    p2r = torch.full((R + 2 * guard,), -7, dtype=torch.int32, device="cuda")
    xp = torch.full((R + 2 * guard, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(max(B.moe_permute_workspace_bytes(d), 16), dtype=torch.uint8, device="cuda")
    assert B.moe_device_status() == 0
    B.moe_permute(d, Hh.to_dev_bf16(X), _i32(idx_np), xp[guard:guard + R], counts[guard:guard + E],
                  offsets[guard:guard + E + 1], r2p[guard:guard + R], p2r[guard:guard + R], ws)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 7                 # MOE_ERR_BAD_INDEX, read once ...
    assert B.moe_device_status() == 0                 # ... and cleared by the read
    # expected: the stable sort of the valid pairs (written out here: the oracle refuses invalid ids)
    vp = np.flatnonzero(valid)
    order = vp[np.argsort(flat[vp], kind="stable")]
    exp_counts = np.bincount(flat[vp], minlength=E)
    exp_p2r = np.full(R, -7, dtype=np.int64)
    exp_p2r[order] = np.arange(n_valid)
    assert np.array_equal(counts[guard:guard + E].cpu().numpy(), exp_counts)
    assert np.array_equal(offsets[guard:guard + E + 1].cpu().numpy(), np.concatenate([[0], np.cumsum(exp_counts)]))
    got_r2p = r2p[guard:guard + R].cpu().numpy()
    assert np.array_equal(got_r2p[:n_valid], order)
    assert np.all(got_r2p[n_valid:] == -7)            # rows past offsets[E] stay unwritten
    assert np.array_equal(p2r[guard:guard + R].cpu().numpy(), exp_p2r)   # dropped pairs keep the sentinel
    rows = Hh.to_np64(xp[guard:guard + R])
    assert np.array_equal(rows[:n_valid], X[order // K].astype(np.float64))
    assert np.all(np.isnan(rows[n_valid:]))
    for t in (counts, offsets, r2p, p2r):              # guard bands untouched
        assert torch.all(t[:guard] == -7) and torch.all(t[-guard:] == -7)
    assert torch.isnan(xp[:guard]).all() and torch.isnan(xp[-guard:]).all()
    # the next ordinary call is unaffected
    _check_permute(B, rng.integers(0, E, size=(T, K)).astype(np.int32), E, X)
    assert B.moe_device_status() == 0


@pytest.mark.parametrize("name", ["fine_grained", "many_small", "few_large", "imbalanced"])
def test_permute_indices_full_size(B, name):
    cfg = W.CONFIGS[name]
    idx, _ = W.make_routing(cfg)
    _check_permute(B, idx, cfg.E)


# ------------------------------------------------------------------------------------------------
# per-call parity (inputs from the oracle chain, rounded to bf16)
# ------------------------------------------------------------------------------------------------
def _dims(B, cfg):
    return B.dims(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K)


def _nan(shape, dtype=torch.bfloat16):
    return torch.full(shape, float("nan"), dtype=dtype, device="cuda")


def test_gateup_swiglu(B, case):
    cfg, host, ref = case
    d, R = _dims(B, cfg), cfg.R
    xp = _r(ref["X_perm"])
    hact, gu = _nan((R, cfg.I)), _nan((R, 2 * cfg.I))
    B.moe_grouped_gemm_gateup_swiglu(d, _bf(xp), _bf(host["W_gate"]), _bf(host["W_up"]), _i32(ref["offsets"]), hact, gu)
    torch.cuda.synchronize()
    o_h, o_gu = O.gateup_swiglu(xp, host["W_gate"], host["W_up"], ref["offsets"])
    Hh.assert_close(Hh.to_np64(gu), o_gu, "GU", rel_fro=Hh.PER_CALL_FROBENIUS)
    Hh.assert_close(Hh.to_np64(hact), o_h, "H_act", rel_fro=Hh.PER_CALL_FROBENIUS)
    # inference form: no saved pre-activations
    hact2 = _nan((R, cfg.I))
    B.moe_grouped_gemm_gateup_swiglu(d, _bf(xp), _bf(host["W_gate"]), _bf(host["W_up"]), _i32(ref["offsets"]), hact2, None)
    torch.cuda.synchronize()
    assert torch.equal(hact, hact2)


def test_down(B, case):
    cfg, host, ref = case
    d, R = _dims(B, cfg), cfg.R
    h = _r(ref["H_act"])
    yp = _nan((R, cfg.H))
    B.moe_grouped_gemm_down(d, _bf(h), _bf(host["W_down"]), _i32(ref["offsets"]), yp)
    torch.cuda.synchronize()
    Hh.assert_close(Hh.to_np64(yp), O.down(h, host["W_down"], ref["offsets"]), "Y_perm", rel_fro=Hh.PER_CALL_FROBENIUS)


def test_unpermute_combine_and_bwd(B, case):
    cfg, host, ref = case
    d, R = _dims(B, cfg), cfg.R
    yp, dy = _r(ref["Y_perm"]), host["dY"]
    w = torch.from_numpy(host["topk_w"]).cuda()
    p2r = _i32(ref["pair_to_row"])
    y = _nan((cfg.T, cfg.H))
    B.moe_unpermute_combine(d, _bf(yp), w, p2r, y)
    dyp, dw = _nan((R, cfg.H)), _nan((cfg.T, cfg.K), torch.float32)
    B.moe_unpermute_combine_bwd(d, _bf(dy), _bf(yp), w, p2r, dyp, dw)
    dyp2 = _nan((R, cfg.H))
    B.moe_unpermute_combine_bwd(d, _bf(dy), None, w, p2r, dyp2, None)
    torch.cuda.synchronize()
    Hh.assert_close(Hh.to_np64(y), O.unpermute_combine(yp, host["topk_w"], ref["pair_to_row"]), "Y",
                    rel_fro=Hh.PER_CALL_FROBENIUS)
    o_dyp, o_dw = O.unpermute_combine_bwd(dy, yp, host["topk_w"], ref["pair_to_row"])
    Hh.assert_close(Hh.to_np64(dyp), o_dyp, "dY_perm", rel_fro=Hh.PER_CALL_FROBENIUS)
    Hh.assert_close(dw.cpu().numpy().astype(np.float64), o_dw, "dtopk_w", rel_fro=1e-5, max_abs=1e-4)
    assert torch.equal(dyp, dyp2)


def test_down_bwd(B, case):
    cfg, host, ref = case
    d, R = _dims(B, cfg), cfg.R
    dyp, h = _r(ref["dY_perm"]), _r(ref["H_act"])
    dh, dwd = _nan((R, cfg.I)), _nan((cfg.E, cfg.I, cfg.H))
    B.moe_grouped_gemm_down_bwd(d, _bf(dyp), _bf(h), _bf(host["W_down"]), _i32(ref["offsets"]), dh, dwd)
    torch.cuda.synchronize()
    o_dh, o_dwd = O.down_bwd(dyp, h, host["W_down"], ref["offsets"])
    Hh.assert_close(Hh.to_np64(dh), o_dh, "dH_act", rel_fro=Hh.PER_CALL_FROBENIUS)
    Hh.assert_close(Hh.to_np64(dwd), o_dwd, "dW_down", rel_fro=Hh.PER_CALL_FROBENIUS)
    for e in np.flatnonzero(ref["counts"] == 0):
        assert not Hh.to_np64(dwd[e]).any()                 # an expert without rows: exact zeros, written


def test_gateup_swiglu_bwd(B, case):
    cfg, host, ref = case
    d, R = _dims(B, cfg), cfg.R
    dh, gu, xp = _r(ref["dH_act"]), _r(ref["GU"]), _r(ref["X_perm"])
    dgu, dxp = _nan((R, 2 * cfg.I)), _nan((R, cfg.H))
    dwg, dwu = _nan((cfg.E, cfg.H, cfg.I)), _nan((cfg.E, cfg.H, cfg.I))
    B.moe_grouped_gemm_gateup_swiglu_bwd(d, _bf(dh), _bf(gu), _bf(xp), _bf(host["W_gate"]), _bf(host["W_up"]),
                                         _i32(ref["offsets"]), dgu, dxp, dwg, dwu)
    torch.cuda.synchronize()
    o_dgu = O.swiglu_bwd(dh, gu)
    Hh.assert_close(Hh.to_np64(dgu), o_dgu, "dGU", rel_fro=Hh.PER_CALL_FROBENIUS)
    # the GEMMs consume the bf16 dGU the elementwise kernel wrote: same rounding on the oracle side
    o_dxp, o_dwg, o_dwu = O.gateup_bwd_from_dgu(_r(o_dgu), xp, host["W_gate"], host["W_up"], ref["offsets"])
    Hh.assert_close(Hh.to_np64(dxp), o_dxp, "dX_perm", rel_fro=3.5e-3)
    Hh.assert_close(Hh.to_np64(dwg), o_dwg, "dW_gate", rel_fro=3.5e-3)
    Hh.assert_close(Hh.to_np64(dwu), o_dwu, "dW_up", rel_fro=3.5e-3)
    for e in np.flatnonzero(ref["counts"] == 0):
        assert not Hh.to_np64(dwg[e]).any() and not Hh.to_np64(dwu[e]).any()


def test_fused_down_dgrad_swiglu_bwd(B, case):
    """The fused entry point against its oracle (inputs from the oracle chain, rounded to bf16), and against the
    two-call form it replaces: the fused result may differ from it only by the rounding of dH_act it avoids."""
    cfg, host, ref = case
    d, R = _dims(B, cfg), cfg.R
    dyp, gu = _r(ref["dY_perm"]), _r(ref["GU"])
    off = _i32(ref["offsets"])
    dgu = _nan((R, 2 * cfg.I))
    B.moe_grouped_gemm_down_dgrad_swiglu_bwd(d, _bf(dyp), _bf(host["W_down"]), _bf(gu), off, dgu)
    torch.cuda.synchronize()
    assert B.moe_device_status() == 0
    o_dgu = O.down_dgrad_swiglu_bwd(dyp, host["W_down"], gu, ref["offsets"])
    Hh.assert_close(Hh.to_np64(dgu), o_dgu, "dGU (fused)", rel_fro=Hh.PER_CALL_FROBENIUS)
    dh, dgu2 = _nan((R, cfg.I)), _nan((R, 2 * cfg.I))
    B.moe_grouped_gemm_down_dgrad(d, _bf(dyp), _bf(host["W_down"]), off, dh)
    B.moe_swiglu_bwd(d, dh, _bf(gu), dgu2)
    torch.cuda.synchronize()
    two = Hh.error_stats(Hh.to_np64(dgu2), o_dgu)
    one = Hh.error_stats(Hh.to_np64(dgu), o_dgu)
    assert one["rel_fro"] <= two["rel_fro"] * 1.02, (one, two)      # one rounding fewer: never worse


def test_gateup_pieces_from_given_dgu(B, case):
    """dgrad and wgrad alone, fed the oracle's dGU: isolates the two GEMMs from the elementwise kernel."""
    cfg, host, ref = case
    d, R = _dims(B, cfg), cfg.R
    dgu, xp = _r(ref["dGU"]), _r(ref["X_perm"])
    dxp = _nan((R, cfg.H))
    dwg, dwu = _nan((cfg.E, cfg.H, cfg.I)), _nan((cfg.E, cfg.H, cfg.I))
    B.moe_grouped_gemm_gateup_dgrad(d, _bf(dgu), _bf(host["W_gate"]), _bf(host["W_up"]), _i32(ref["offsets"]), dxp)
    B.moe_grouped_gemm_gateup_wgrad(d, _bf(xp), _bf(dgu), _i32(ref["offsets"]), dwg, dwu)
    torch.cuda.synchronize()
    o_dxp, o_dwg, o_dwu = O.gateup_bwd_from_dgu(dgu, xp, host["W_gate"], host["W_up"], ref["offsets"])
    Hh.assert_close(Hh.to_np64(dxp), o_dxp, "dX_perm", rel_fro=Hh.PER_CALL_FROBENIUS)
    Hh.assert_close(Hh.to_np64(dwg), o_dwg, "dW_gate", rel_fro=Hh.PER_CALL_FROBENIUS)
    Hh.assert_close(Hh.to_np64(dwu), o_dwu, "dW_up", rel_fro=Hh.PER_CALL_FROBENIUS)


def test_permute_bwd(B, case):
    cfg, host, ref = case
    d = _dims(B, cfg)
    dxp = _r(ref["dX_perm"])
    dx = _nan((cfg.T, cfg.H))
    B.moe_permute_bwd(d, _bf(dxp), _i32(ref["pair_to_row"]), dx)
    torch.cuda.synchronize()
    Hh.assert_close(Hh.to_np64(dx), O.permute_bwd(dxp, ref["pair_to_row"], cfg.T, cfg.K), "dX",
                    rel_fro=Hh.PER_CALL_FROBENIUS)


# ------------------------------------------------------------------------------------------------
# end to end: the CUDA chain against the unrounded fp64 chain; determinism; guard bands
# ------------------------------------------------------------------------------------------------
FLOAT_OUTPUTS = [("y", "Y"), ("dx", "dX"), ("dw_gate", "dW_gate"), ("dw_up", "dW_up"), ("dw_down", "dW_down"),
                 ("h_act", "H_act"), ("gu", "GU"), ("y_perm", "Y_perm"), ("dy_perm", "dY_perm"), ("dh_act", "dH_act"),
                 ("dgu", "dGU"), ("dx_perm", "dX_perm")]


def test_end_to_end_exact_chain(B, case):
    cfg, host, ref = case
    dev = Hh.device_workload(host)
    b = Hh.run_cuda_layer(dev, cfg.E)
    for name in ("counts", "offsets", "row_to_pair", "pair_to_row"):
        assert np.array_equal(getattr(b, name).cpu().numpy(), ref[name]), name
    for attr, key in FLOAT_OUTPUTS:
        Hh.assert_close(Hh.to_np64(getattr(b, attr)), ref[key], key)
    Hh.assert_close(b.dtopk_w.cpu().numpy().astype(np.float64), ref["dtopk_w"], "dtopk_w")


def test_bitwise_determinism(B, case):
    cfg, host, ref = case
    dev = Hh.device_workload(host)
    b1 = Hh.run_cuda_layer(dev, cfg.E)
    b2 = Hh.run_cuda_layer(dev, cfg.E)
    for attr, _ in FLOAT_OUTPUTS + [("dtopk_w", ""), ("row_to_pair", ""), ("pair_to_row", "")]:
        assert torch.equal(getattr(b1, attr), getattr(b2, attr)), attr


def test_rows_past_the_last_expert_row_and_guard_bands_untouched(B):
    """Outputs are allocated with a sentinel band before and after; nothing outside the tensor may
    be written (stands in for a memory checker)."""
    cfg, host = Hh.ragged_workload([3, 0, 130, 123], K=2, H=128, I=128, seed=3)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"],
                          host["W_down"], host["dY"])
    d, R = _dims(B, cfg), cfg.R
    pad = 4096

    def banded(rows, cols):
        buf = torch.full((pad + rows * cols + pad,), 123.0, dtype=torch.bfloat16, device="cuda")
        return buf, buf[pad:pad + rows * cols].view(rows, cols)

    xp, off = _bf(_r(ref["X_perm"])), _i32(ref["offsets"])
    hb, h = banded(R, cfg.I)
    gb, gu = banded(R, 2 * cfg.I)
    B.moe_grouped_gemm_gateup_swiglu(d, xp, _bf(host["W_gate"]), _bf(host["W_up"]), off, h, gu)
    yb, yp = banded(R, cfg.H)
    B.moe_grouped_gemm_down(d, h, _bf(host["W_down"]), off, yp)
    wb, dwd = banded(cfg.E * cfg.I, cfg.H)
    B.moe_grouped_gemm_down_wgrad(d, h, _bf(_r(ref["dY_perm"])), off, dwd)
    torch.cuda.synchronize()
    for buf in (hb, gb, yb, wb):
        assert torch.all(buf[:pad] == 123.0) and torch.all(buf[-pad:] == 123.0)
    Hh.assert_close(Hh.to_np64(yp), O.down(Hh.to_np64(h), host["W_down"], ref["offsets"]), "Y_perm",
                    rel_fro=Hh.PER_CALL_FROBENIUS)


def test_unit_weight_identities(B):
    """K=1: permute then unpermute with unit weights is the identity, bit for bit; K=4 with w=1/4 too."""
    rng = np.random.default_rng(0)
    T, H, E = 300, 256, 7
    X = W.round_to_bf16(rng.standard_normal((T, H)).astype(np.float32))
    for K, wv in ((1, 1.0), (4, 0.25)):
        idx = np.argsort(rng.standard_normal((T, E)), axis=1)[:, :K].astype(np.int32)
        b = B.alloc_layer_buffers(T, H, 128, E, K)
        x = Hh.to_dev_bf16(X)
        B.moe_permute(b.d, x, _i32(idx), b.x_perm, b.counts, b.offsets, b.row_to_pair, b.pair_to_row, b.workspace)
        w = torch.full((T, K), wv, dtype=torch.float32, device="cuda")
        B.moe_unpermute_combine(b.d, b.x_perm, w, b.pair_to_row, b.y)
        torch.cuda.synchronize()
        assert torch.equal(b.y, x)


def test_host_entry_point_matches_device_chain(B):
    cfg = W.CONFIGS["tiny"]
    host = W.make_workload(cfg)
    dev = Hh.device_workload(host)
    b = Hh.run_cuda_layer(dev, cfg.E)
    d = _dims(B, cfg)
    arena = torch.empty(B.moe_layer_arena_bytes(d), dtype=torch.uint8, device="cuda")
    pin = lambda t: t.cpu().pin_memory()
    xh, ih, wh, dyh = pin(dev["X"]), pin(dev["topk_idx"]), pin(dev["topk_w"]), pin(dev["dY"])
    yh = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16).pin_memory()
    dxh = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16).pin_memory()
    dwh = torch.empty((cfg.T, cfg.K), dtype=torch.float32).pin_memory()
    dwg, dwu, dwd = torch.empty_like(b.dw_gate), torch.empty_like(b.dw_up), torch.empty_like(b.dw_down)
    # three calls back to back without host synchronisation in between (the internal copy stream and its
    # events are reused): the last one must still give the device chain's results
    for _ in range(3):
        B.moe_layer_fwd_bwd_host(d, xh, ih, wh, dyh, dev["W_gate"], dev["W_up"], dev["W_down"], yh, dxh, dwh, dwg, dwu, dwd,
                                 arena)
    torch.cuda.synchronize()
    assert torch.equal(yh, b.y.cpu()) and torch.equal(dxh, b.dx.cpu()) and torch.equal(dwh, b.dtopk_w.cpu())
    assert torch.equal(dwg, b.dw_gate) and torch.equal(dwu, b.dw_up) and torch.equal(dwd, b.dw_down)
    # different inputs through the same arena: exact scaling by a power of two
    xh2, dyh2 = (xh.float() * 2).to(torch.bfloat16).pin_memory(), (dyh.float() * 0.5).to(torch.bfloat16).pin_memory()
    B.moe_layer_fwd_bwd_host(d, xh2, ih, wh, dyh2, dev["W_gate"], dev["W_up"], dev["W_down"], yh, dxh, dwh, dwg, dwu, dwd,
                             arena)
    torch.cuda.synchronize()
    dev2 = dict(dev, X=xh2.cuda(), dY=dyh2.cuda())
    b2 = Hh.run_cuda_layer(dev2, cfg.E)
    assert torch.equal(yh, b2.y.cpu()) and torch.equal(dxh, b2.dx.cpu()) and torch.equal(dwh, b2.dtopk_w.cpu())
    assert torch.equal(dwg, b2.dw_gate) and torch.equal(dwd, b2.dw_down)


def test_host_entry_point_pipelines_different_steps(B):
    """Four calls in a row, each with its own host inputs, routing and host outputs, no synchronisation in between:
    the uploads of a call run under the previous call's backward pass, and every call must still give exactly
    the device chain's results for ITS inputs (a stress of the event ordering around the shared arena)."""
    cfg, base = Hh.ragged_workload([600, 540, 0, 700], K=2, H=320, I=192, seed=11)   # large enough to overlap for real
    d = _dims(B, cfg)
    arena = torch.empty(B.moe_layer_arena_bytes(d), dtype=torch.uint8, device="cuda")
    dev0 = Hh.device_workload(base)
    pin = lambda t: t.cpu().pin_memory()
    rng = np.random.default_rng(3)
    steps = []
    for i in range(4):
        scale = float(2.0 ** (i - 1))
        x = (dev0["X"].float() * scale).to(torch.bfloat16)
        dy = (dev0["dY"].float() / scale).to(torch.bfloat16)
        idx = dev0["topk_idx"].cpu().numpy().copy()
        if i % 2:                                        # another routing on odd steps: expert ids mirrored
            idx = (cfg.E - 1 - idx).astype(np.int32)
        dev = dict(dev0, X=x, dY=dy, topk_idx=torch.from_numpy(idx).cuda())
        out = dict(y=torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16).pin_memory(),
                   dx=torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16).pin_memory(),
                   dw=torch.empty((cfg.T, cfg.K), dtype=torch.float32).pin_memory(),
                   dwg=torch.empty_like(dev0["W_gate"]), dwu=torch.empty_like(dev0["W_up"]),
                   dwd=torch.empty_like(dev0["W_down"]))
        steps.append((dev, dict(x=pin(x), idx=pin(dev["topk_idx"]), w=pin(dev["topk_w"]), dy=pin(dy)), out))
    for dev, h, o in steps:
        B.moe_layer_fwd_bwd_host(d, h["x"], h["idx"], h["w"], h["dy"], dev["W_gate"], dev["W_up"], dev["W_down"],
                                 o["y"], o["dx"], o["dw"], o["dwg"], o["dwu"], o["dwd"], arena)
    torch.cuda.synchronize()
    for dev, h, o in steps:
        b = Hh.run_cuda_layer(dev, cfg.E)
        assert torch.equal(o["y"], b.y.cpu()) and torch.equal(o["dx"], b.dx.cpu()) and torch.equal(o["dw"], b.dtopk_w.cpu())
        assert torch.equal(o["dwg"], b.dw_gate) and torch.equal(o["dwu"], b.dw_up) and torch.equal(o["dwd"], b.dw_down)


# ------------------------------------------------------------------------------------------------
# degenerate shapes: a single expert, top-1, fewer rows than one tile, one token, many experts
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T,H,I,E,K", [(1, 128, 128, 1, 1), (3, 128, 128, 4, 2), (130, 256, 128, 1, 1),
                                       (64, 128, 256, 300, 4), (40, 384, 128, 33, 32), (513, 128, 128, 2, 1),
                                       (70, 64, 64, 3, 2), (700, 64, 192, 2, 2), (1200, 192, 64, 2, 1),    # smallest H, I
                                       (1500, 128, 128, 1024, 2)])                                         # most experts
def test_degenerate_shapes_end_to_end(B, T, H, I, E, K):
    cfg = W.MoeConfig("deg", T=T, H=H, I=I, E=E, K=K, routing="softmax", cfg_id=70 + T % 7)
    host = W.make_workload(cfg)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"],
                          host["W_down"], host["dY"])
    b = Hh.run_cuda_layer(Hh.device_workload(host), E)
    for name in ("counts", "offsets", "row_to_pair", "pair_to_row"):
        assert np.array_equal(getattr(b, name).cpu().numpy(), ref[name]), name
    for attr, key in FLOAT_OUTPUTS:
        Hh.assert_close(Hh.to_np64(getattr(b, attr)), ref[key], key)
    Hh.assert_close(b.dtopk_w.cpu().numpy().astype(np.float64), ref["dtopk_w"], "dtopk_w")


def test_pair_and_single_tile_shapes_agree(B):
    """The same experts' rows run through the CTA-pair kernels (>= 512 rows per expert on average) and, split
    over twice as many experts with duplicated weights, through the single-CTA kernels: equal outputs."""
    counts = [700, 650, 520, 690]
    cfg, host = Hh.ragged_workload(counts, K=2, H=256, I=256, seed=5)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"],
                          host["W_down"], host["dY"])
    b = Hh.run_cuda_layer(Hh.device_workload(host), cfg.E)            # 640 rows per expert: pair kernels
    for attr, key in FLOAT_OUTPUTS:
        Hh.assert_close(Hh.to_np64(getattr(b, attr)), ref[key], key)
    # pad with 4 experts that get no rows: 320 rows per expert on average -> single-CTA kernels
    pad = lambda w: np.concatenate([w, np.zeros_like(w)], axis=0)
    host2 = dict(host, W_gate=pad(host["W_gate"]), W_up=pad(host["W_up"]), W_down=pad(host["W_down"]))
    b2 = Hh.run_cuda_layer(Hh.device_workload(host2), 2 * cfg.E)
    for attr in ("y", "dx", "h_act", "gu", "y_perm", "dh_act", "dgu", "dx_perm"):
        assert torch.equal(getattr(b, attr), getattr(b2, attr)), attr   # same arithmetic order per element
    for attr in ("dw_gate", "dw_up", "dw_down"):
        assert torch.equal(getattr(b, attr), getattr(b2, attr)[:cfg.E]), attr
        assert not bool(getattr(b2, attr)[cfg.E:].any())


def test_layer_can_be_captured_in_a_cuda_graph_and_replayed(B):
    """All work is enqueued on the caller's stream with no host synchronisation or allocation, so a whole
    forward + backward can be captured once and replayed on new inputs written into the same buffers."""
    cfg, host = Hh.ragged_workload([300, 0, 77, 200, 1, 190], K=2, H=256, I=256, seed=7)
    dev = Hh.device_workload(host)
    b = Hh.run_cuda_layer(dev, cfg.E)                       # first calls (attribute set-up) outside capture
    want = {a: getattr(b, a).clone() for a, _ in FLOAT_OUTPUTS}
    x_static, dy_static = dev["X"].clone(), dev["dY"].clone()
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            B.layer_forward(b, x_static, dev["topk_idx"], dev["topk_w"], dev["W_gate"], dev["W_up"], dev["W_down"])
            B.layer_backward(b, dy_static, dev["topk_w"], dev["W_gate"], dev["W_up"], dev["W_down"])
    for a, _ in FLOAT_OUTPUTS:
        getattr(b, a).fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    for a, _ in FLOAT_OUTPUTS:
        assert torch.equal(getattr(b, a), want[a]), a
    # new inputs in the captured buffers: doubling X and dY doubles X_perm and dY_perm exactly (powers of two)
    x_static.mul_(2.0)
    dy_static.mul_(2.0)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(b.x_perm, want["x_perm"] * 2) if "x_perm" in want else True
    assert torch.equal(b.dy_perm, want["dy_perm"] * 2)
    assert B.moe_device_status() == 0
