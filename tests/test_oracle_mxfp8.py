"""Pins of the oracle's block-scaled FP8 (MXFP8: E4M3 elements, E8M0 scale per 32 elements) quantiser and of the
quantised down projection, against what the format definition and the mathematics fix."""
import numpy as np
import torch

from oracle import moe_oracle as O


def test_all_e4m3_codes_round_trip_and_match_the_library_type():
    codes = np.arange(256, dtype=np.uint8)
    vals = O.e4m3_decode(codes)
    finite = ~np.isnan(vals)
    assert (~finite).sum() == 2 and np.isnan(vals[0x7F]) and np.isnan(vals[0xFF])
    assert vals[0x7E] == 448.0 and vals[0x01] == 2.0 ** -9 and vals[0x08] == 2.0 ** -6 and vals[0x38] == 1.0
    # decode agrees with torch's float8_e4m3fn bit pattern interpretation
    lib = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(vals[finite], lib[finite])
    # every representable value encodes to its own code (negative zero keeps its sign bit)
    back = O.e4m3_encode(vals[finite])
    assert np.array_equal(back, codes[finite])


def test_e4m3_encode_rounds_to_nearest_even_and_saturates():
    # halfway between 1.0 (mantissa 000, even) and 1.125 (001): ties to 1.0; between 1.125 and 1.25 (010): to 1.25
    assert O.e4m3_decode(O.e4m3_encode([1.0625, 1.1875, -1.0625]))[...].tolist() == [1.0, 1.25, -1.0]
    # just above / below a halfway point
    assert O.e4m3_decode(O.e4m3_encode([1.0625 + 1e-9, 1.1875 - 1e-9])).tolist() == [1.125, 1.125]
    # subnormal grid 2^-9: 1.5 * 2^-9 ties to even (2 * 2^-9), 0.5 * 2^-9 ties to zero
    assert O.e4m3_decode(O.e4m3_encode([1.5 * 2.0 ** -9, 0.5 * 2.0 ** -9, 0.75 * 2.0 ** -9])).tolist() == [2.0 ** -8, 0.0, 2.0 ** -9]
    # saturation instead of NaN/inf; 464 is halfway between 448 and the (non-existent) 480
    assert O.e4m3_decode(O.e4m3_encode([449.0, 464.0, 500.0, 1e9, -1e9])).tolist() == [448.0, 448.0, 448.0, 448.0, -448.0]
    # in range, the library cast (round to nearest even) gives the same codes
    rng = np.random.default_rng(0)
    y = np.concatenate([rng.uniform(-440, 440, 4000), rng.standard_normal(4000) * 0.01, rng.standard_normal(4000)])
    lib = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = O.e4m3_encode(y)
    nz = O.e4m3_decode(got) != 0          # the sign of a value that rounds to zero is the one place conventions may differ
    assert np.array_equal(got[nz], lib[nz])


def test_scale_selection_on_hand_built_blocks():
    blk = np.zeros((5, 32))
    blk[0, 3] = 1.0            # amax 1 = 2^0        -> scale 2^-8, code of 256 = 1.0 * 2^8
    blk[1, 7] = -447.9         # amax in [256, 512)  -> scale 2^0
    blk[2, :] = 3.0e-5         # amax 3e-5 ~ 1.97 * 2^-16 -> floor(log2) = -16 -> scale 2^-24
    blk[3, 0] = 500.0          # amax 500 -> floor(log2) = 8 -> scale 2^0: 500 saturates to 448
    # row 4 stays all zero
    codes, scales, deq = O.mxfp8_quantize(blk)
    assert scales[:, 0].tolist() == [127 - 8, 127, 127 - 24, 127, 0]
    assert deq[0, 3] == 1.0 and codes[0, 3] == O.e4m3_encode([256.0])[0]
    assert deq[1, 7] == -448.0
    assert deq[3, 0] == 448.0
    assert not codes[4].any() and not deq[4].any()
    # the largest element of a block always lands in [256, 512) before rounding: top binade, never a subnormal
    rng = np.random.default_rng(1)
    x = rng.standard_normal((64, 96)) * np.exp2(rng.integers(-20, 20, size=(64, 1)))
    codes, scales, deq = O.mxfp8_quantize(x)
    top = np.max(np.abs(O.e4m3_decode(codes)).reshape(64, 3, 32), axis=-1)
    assert np.all((top >= 256.0) & (top <= 448.0))
    # scales are per block of 32 along the last axis and nothing else
    assert scales.shape == (64, 3)
    c2, s2, d2 = O.mxfp8_quantize(x[:, 32:64])
    assert np.array_equal(c2, codes[:, 32:64]) and np.array_equal(s2[:, 0], scales[:, 1])


def test_quantisation_error_bound_and_idempotence():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((200, 128))
    codes, scales, deq = O.mxfp8_quantize(x)
    scale = np.exp2(scales.astype(np.float64) - 127.0).repeat(32, axis=1)
    # elements that stay normal after scaling (|v| >= 2^-6 * scale): relative error at most half an ulp = 2^-4;
    # the rest: absolute error at most half the subnormal spacing; saturated top elements: below 512 -> 448, 12.5 %
    normal = np.abs(x) >= 2.0 ** -6 * scale
    sat = np.abs(x) / scale > 448.0
    assert np.all(np.abs(deq - x)[normal & ~sat] <= 2.0 ** -4 * np.abs(x)[normal & ~sat] * (1 + 1e-12))
    assert np.all(np.abs(deq - x)[~normal] <= 2.0 ** -10 * scale[~normal] * (1 + 1e-12))
    assert np.all(np.abs(deq - x)[sat] <= 0.125 * np.abs(x)[sat])
    # quantising the dequantised values changes nothing (they are representable with the same scales)
    c2, s2, d2 = O.mxfp8_quantize(deq)
    assert np.array_equal(c2, codes) and np.array_equal(s2, scales) and np.array_equal(d2, deq)
    # typical size of the error of a Gaussian block: a few per cent, far above bf16's 2^-9
    rel = np.linalg.norm(deq - x) / np.linalg.norm(x)
    assert 0.015 < rel < 0.04


def test_down_mxfp8_is_the_exact_product_of_the_dequantised_operands():
    rng = np.random.default_rng(3)
    E, I, H = 3, 64, 24
    counts = [5, 0, 9]
    offsets = np.concatenate([[0], np.cumsum(counts)])
    Hact = rng.standard_normal((14, I))
    Wd = rng.standard_normal((E, I, H)) * 0.05
    got = O.down_mxfp8(Hact, Wd, offsets)
    # written out per element with the quantiser applied by hand to each operand vector
    for r, e in ((0, 0), (4, 0), (5, 2), (13, 2)):
        a = O.mxfp8_quantize(Hact[r])[2]
        for h in (0, 7, 23):
            b = O.mxfp8_quantize(Wd[e, :, h])[2]          # the weight column's own scales along I
            assert abs(got[r, h] - float(a @ b)) <= 1e-12
    # against the unquantised product: a few per cent, and exactly equal when the operands are representable
    ref = O.down(Hact, Wd, offsets)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert 0.01 < rel < 0.06
    Hq = O.mxfp8_quantize(Hact)[2]
    Wq = np.swapaxes(O.mxfp8_quantize(np.swapaxes(Wd, 1, 2))[2], 1, 2)
    assert np.array_equal(O.down_mxfp8(Hq, Wq, offsets), O.down(Hq, Wq, offsets))


def test_down_dgrad_mxfp8_is_the_exact_product_of_the_dequantised_operands():
    rng = np.random.default_rng(4)
    E, I, H = 3, 64, 96
    counts = [0, 6, 7]
    offsets = np.concatenate([[0], np.cumsum(counts)])
    dYp = rng.standard_normal((13, H))
    Wd = rng.standard_normal((E, I, H)) * 0.05
    got = O.down_dgrad_mxfp8(dYp, Wd, offsets)
    assert got.shape == (13, I)
    # written out per element with the quantiser applied by hand to each operand vector (both along H)
    for r, e in ((0, 1), (5, 1), (6, 2), (12, 2)):
        a = O.mxfp8_quantize(dYp[r])[2]
        for i in (0, 9, 19):
            b = O.mxfp8_quantize(Wd[e, i, :])[2]
            assert abs(got[r, i] - float(a @ b)) <= 1e-12
    # against the unquantised data gradient: a few per cent; exactly equal when the operands are representable
    ref = O.down_bwd(dYp, rng.standard_normal((13, I)), Wd, offsets)[0]
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert 0.01 < rel < 0.06
    dq, wq = O.mxfp8_quantize(dYp)[2], O.mxfp8_quantize(Wd)[2]
    assert np.array_equal(O.down_dgrad_mxfp8(dq, wq, offsets), O.down_bwd(dq, np.zeros((13, I)), wq, offsets)[0])
    # a transposed weight operand (scales taken along I instead of H) is a different, detectably different, result
    wrong = np.zeros_like(got)
    w_alt = np.swapaxes(O.mxfp8_quantize(np.swapaxes(Wd, 1, 2))[2], 1, 2)
    for e in range(E):
        lo, hi = offsets[e], offsets[e + 1]
        wrong[lo:hi] = O.mxfp8_quantize(dYp)[2][lo:hi] @ w_alt[e].T
    assert np.abs(wrong - got).max() > 1e-6


def test_gateup_dgrad_mxfp8_is_the_exact_product_of_the_dequantised_operands():
    rng = np.random.default_rng(5)
    E, I, H = 2, 64, 12
    counts = [4, 7]
    offsets = np.concatenate([[0], np.cumsum(counts)])
    dGU = rng.standard_normal((11, 2 * I)) * np.concatenate([np.full(I, 1.0), np.full(I, 37.0)])   # halves of different size
    Wg = rng.standard_normal((E, H, I)) * 0.05
    Wu = rng.standard_normal((E, H, I)) * 0.3
    got = O.gateup_dgrad_mxfp8(dGU, Wg, Wu, offsets)
    assert got.shape == (11, H)
    for r, e in ((0, 0), (3, 0), (4, 1), (10, 1)):
        ag = O.mxfp8_quantize(dGU[r, :I])[2]
        au = O.mxfp8_quantize(dGU[r, I:])[2]
        for h in (0, 5, 11):
            bg = O.mxfp8_quantize(Wg[e, h, :])[2]
            bu = O.mxfp8_quantize(Wu[e, h, :])[2]
            assert abs(got[r, h] - float(ag @ bg + au @ bu)) <= 1e-10
    # against the unquantised data gradient (the bf16 path's own oracle): a few per cent; equal for representable operands
    ref = O.gateup_bwd_from_dgu(dGU, np.zeros((11, H)), Wg, Wu, offsets)[0]
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert 0.01 < rel < 0.06
    dq, gq, uq = O.mxfp8_quantize(dGU)[2], O.mxfp8_quantize(Wg)[2], O.mxfp8_quantize(Wu)[2]
    assert np.allclose(O.gateup_dgrad_mxfp8(dq, gq, uq, offsets), O.gateup_bwd_from_dgu(dq, np.zeros((11, H)), gq, uq, offsets)[0],
                       rtol=0, atol=1e-12)
    # swapping the two weight operands is a different result
    assert np.abs(O.gateup_dgrad_mxfp8(dGU, Wu, Wg, offsets) - got).max() > 1e-3


def test_gateup_mxfp8_is_the_exact_product_of_the_dequantised_operands_and_swiglu_fwd_its_activation():
    rng = np.random.default_rng(6)
    E, I, H = 2, 10, 96
    counts = [5, 8]
    offsets = np.concatenate([[0], np.cumsum(counts)])
    Xp = rng.standard_normal((13, H))
    Wg = rng.standard_normal((E, H, I)) * 0.05
    Wu = rng.standard_normal((E, H, I)) * 0.4
    got = O.gateup_mxfp8(Xp, Wg, Wu, offsets)
    assert got.shape == (13, 2 * I)
    for r, e in ((0, 0), (4, 0), (5, 1), (12, 1)):
        a = O.mxfp8_quantize(Xp[r])[2]
        for i in (0, 3, 9):
            assert abs(got[r, i] - float(a @ O.mxfp8_quantize(Wg[e, :, i])[2])) <= 1e-12        # gate column's own scales along H
            assert abs(got[r, I + i] - float(a @ O.mxfp8_quantize(Wu[e, :, i])[2])) <= 1e-12
    # against the unquantised projection: a few per cent; equal for representable operands
    h_ref, gu_ref = O.gateup_swiglu(Xp, Wg, Wu, offsets)
    rel = np.linalg.norm(got - gu_ref) / np.linalg.norm(gu_ref)
    assert 0.01 < rel < 0.06
    xq = O.mxfp8_quantize(Xp)[2]
    gq = np.swapaxes(O.mxfp8_quantize(np.swapaxes(Wg, 1, 2))[2], 1, 2)
    uq = np.swapaxes(O.mxfp8_quantize(np.swapaxes(Wu, 1, 2))[2], 1, 2)
    assert np.array_equal(O.gateup_mxfp8(xq, gq, uq, offsets), O.gateup_swiglu(xq, gq, uq, offsets)[1])
    # the activation of given pre-activations: the pinned forward's own H_act, and closed forms
    assert np.array_equal(O.swiglu_fwd(gu_ref), h_ref)
    assert np.allclose(O.swiglu_fwd(np.array([[0.0, 2.0, -2.0, 5.0, 7.0, 7.0]])), [[0.0, 2.0 / (1 + np.exp(-2.0)) * 7.0, -2.0 / (1 + np.exp(2.0)) * 7.0]])
    t = torch.tensor(gu_ref)
    assert np.allclose(O.swiglu_fwd(gu_ref), (torch.nn.functional.silu(t[:, :I]) * t[:, I:]).numpy(), rtol=1e-12, atol=1e-14)


def test_wgrad_mxfp8_quantises_columns_in_expert_aligned_row_blocks():
    rng = np.random.default_rng(7)
    E, M, N = 4, 6, 5
    counts = [40, 0, 32, 7]                       # a short last block, an empty expert, a whole block, less than a block
    offsets = np.concatenate([[0], np.cumsum(counts)])
    R = int(offsets[-1])
    A = rng.standard_normal((R, M)) * np.exp2(rng.integers(-6, 6, size=(R, 1)))     # rows of very different size
    B = rng.standard_normal((R, N))
    got = O.wgrad_mxfp8(A, B, offsets)
    assert got.shape == (E, M, N) and not got[1].any()
    # by hand: expert 0 has the row blocks [0,32) and [32,40); expert 3 the block [72,79)
    def col(x, lo, hi):                            # one column segment quantised as its own (zero-padded) block
        seg = np.zeros(32)
        seg[:hi - lo] = x[lo:hi]
        return O.mxfp8_quantize(seg)[2][:hi - lo]
    for (e, blocks) in ((0, [(0, 32), (32, 40)]), (2, [(40, 72)]), (3, [(72, 79)])):
        for m in (0, 5):
            for n in (0, 4):
                want = sum(float(col(A[:, m], lo, hi) @ col(B[:, n], lo, hi)) for lo, hi in blocks)
                assert abs(got[e, m, n] - want) <= 1e-10
    # against the unquantised weight gradient (the bf16 path's own pinned oracle): a few per cent; equal for representable data
    ref = O.down_bwd(B, A, np.zeros((E, M, N)), offsets)[1]          # dWd[e] = Hact_e^T dYp_e with Hact = A, dYp = B
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert 0.01 < rel < 0.08
    Aq, Bq = np.zeros_like(A), np.zeros_like(B)
    for e in range(E):                             # make both operands representable in the same blocks
        lo, hi = offsets[e], offsets[e + 1]
        for b0 in range(lo, hi, 32):
            b1 = min(b0 + 32, hi)
            for x, xq in ((A, Aq), (B, Bq)):
                for c in range(x.shape[1]):
                    xq[b0:b1, c] = col(x[:, c], b0, b1)
    assert np.allclose(O.wgrad_mxfp8(Aq, Bq, offsets), O.down_bwd(Bq, Aq, np.zeros((E, M, N)), offsets)[1], rtol=0, atol=1e-12)
    # the blocks are counted from the expert's first row, not from row 0 of the packed array: moving all rows by 8 changes nothing
    shifted = np.concatenate([[0], np.cumsum([40, 0, 32, 7])])
    A2, B2 = np.concatenate([np.zeros((8, M)), A]), np.concatenate([np.zeros((8, N)), B])     # same rows, moved by 8
    assert np.allclose(O.wgrad_mxfp8(A2, B2, shifted + 8)[[0, 2, 3]], got[[0, 2, 3]])
