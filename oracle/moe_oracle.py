"""Plain fp64 CPU oracle for the MoE expert-FFN hot path (forward and backward).

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of what the
CUDA library computes.  It shares no code with the CUDA path and must never be imported by the
product package; only the tests, the smoke check and the CPU-baseline leg of the benchmark call it.

Every function takes numpy arrays (any float dtype holding the exact input values, e.g. float32
arrays whose values are bf16-representable), converts them to float64 and evaluates the plain
mathematical definition with no intermediate rounding.  A library matmul / stable sort is used as
a step; there is no blocking, fusion or reordering beyond the per-expert loop the packed layout
itself implies.

Notation: T tokens, H hidden, I per-expert intermediate, E experts, K = top-k, R = T*K routed rows.
Pair id p = t*K + k (token-major).  Rows of the packed buffers are ordered by expert; the
per-expert row ranges are [offsets[e], offsets[e+1]).

What each step follows:
  * packed-by-expert buffer + cumulative row counts: the paper's appendix on the dW1 kernel
    ("What the kernel computes"); its inclusive cumulative-sum vector equals offsets[1:].
  * weight gradient of the first projection, dW1_e = X_e^T G_e with G_e the gradient of the
    pre-activation: the paper's section "Production Validation: VeOmni MoE" and the same appendix.
  * an expert with no rows gets an all-zero weight-gradient tile: same appendix (routing model
    paragraph, empty experts K_e = 0).
  * everything else (SwiGLU, down projection, weighted combine, the remaining gradients): the
    standard MoE FFN algebra and the chain rule.

Pins (tests/test_oracle_*.py): brute-force counting sort, stable-sort library routine, dense
SwiGLU MLP special cases evaluated with an independent library (torch, fp64), per-token loop,
torch.autograd on a per-token formulation, central finite differences, identities of
permute/unpermute, empty-expert zeros; for the router: a per-row selection loop, a library softmax,
shift invariance, the all-ties closed form, finite differences; for the fused down-dgrad + SwiGLU backward:
autograd with respect to the saved pre-activations; for the block-scaled FP8 quantiser: the round trip of all 254
finite codes, a library FP8 cast inside the range, hand-built blocks for the scale choice, ties and saturation,
the half-ulp error bound, idempotence; for the six quantised GEMMs (`gateup_mxfp8`, `down_mxfp8`, `down_dgrad_mxfp8`,
`gateup_dgrad_mxfp8`, `wgrad_mxfp8`) and `swiglu_fwd`: per-element products with the quantiser applied by hand to each
operand vector (expert-aligned row blocks for the weight gradients), equality with the pinned bf16-path function on
representable operands, detectably different results for a transposed or swapped operand, a library SiLU.  No function
here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _f64(a):
    return np.asarray(a).astype(F64, copy=False)


# --------------------------------------------------------------------------------------------
# O1  route-permute: stable sort of (token, slot) pairs by expert
# --------------------------------------------------------------------------------------------
def permute_indices(topk_idx, E):
    """counts[E], offsets[E+1] (exclusive prefix, offsets[E]=R), row_to_pair[R], pair_to_row[R].

    row_to_pair lists the pair ids p = t*K+k sorted by (expert(p), p): a stable sort by expert.
    All int32.  The paper's inclusive cumulative-sum vector is offsets[1:].
    """
    idx = np.asarray(topk_idx)
    e_of_p = idx.reshape(-1).astype(np.int64)
    R = e_of_p.size
    if R and (e_of_p.min() < 0 or e_of_p.max() >= E):
        raise ValueError("expert id out of range")
    counts = np.bincount(e_of_p, minlength=E).astype(np.int64)
    offsets = np.zeros(E + 1, dtype=np.int64)
    offsets[1:] = np.cumsum(counts)
    row_to_pair = np.argsort(e_of_p, kind="stable")
    pair_to_row = np.empty(R, dtype=np.int64)
    pair_to_row[row_to_pair] = np.arange(R, dtype=np.int64)
    return (counts.astype(np.int32), offsets.astype(np.int32),
            row_to_pair.astype(np.int32), pair_to_row.astype(np.int32))


def permute(X, topk_idx, E):
    """X_perm[r,:] = X[row_to_pair[r] // K, :] plus the index arrays of permute_indices."""
    X = _f64(X)
    K = np.asarray(topk_idx).shape[1]
    counts, offsets, row_to_pair, pair_to_row = permute_indices(topk_idx, E)
    X_perm = X[row_to_pair.astype(np.int64) // K, :]
    return X_perm, counts, offsets, row_to_pair, pair_to_row


# --------------------------------------------------------------------------------------------
# O2  grouped GEMM gate/up + SwiGLU
# --------------------------------------------------------------------------------------------
def gateup_swiglu(X_perm, W_gate, W_up, offsets):
    """For rows r of expert e: g = Xp[r] @ Wg[e], u = Xp[r] @ Wu[e]; Hact = silu(g)*u.

    Returns Hact [R,I] and the saved pre-activations GU [R,2I] = [g | u].
    silu(g) = g / (1 + exp(-g)).
    """
    Xp = _f64(X_perm)
    E, H, I = W_gate.shape
    R = Xp.shape[0]
    Hact = np.zeros((R, I), F64)
    GU = np.zeros((R, 2 * I), F64)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        g = Xp[r0:r1] @ _f64(W_gate[e])
        u = Xp[r0:r1] @ _f64(W_up[e])
        GU[r0:r1, :I] = g
        GU[r0:r1, I:] = u
        Hact[r0:r1] = g / (1.0 + np.exp(-g)) * u
    return Hact, GU


# --------------------------------------------------------------------------------------------
# O3  grouped GEMM down
# --------------------------------------------------------------------------------------------
def down(H_act, W_down, offsets):
    """Yp[r,:] = Hact[r,:] @ Wd[e] for rows r of expert e."""
    Hact = _f64(H_act)
    E, I, H = W_down.shape
    Yp = np.zeros((Hact.shape[0], H), F64)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 > r0:
            Yp[r0:r1] = Hact[r0:r1] @ _f64(W_down[e])
    return Yp


# --------------------------------------------------------------------------------------------
# O4  unpermute-combine
# --------------------------------------------------------------------------------------------
def unpermute_combine(Y_perm, topk_w, pair_to_row):
    """Y[t,:] = sum_k w[t,k] * Yp[pair_to_row[t*K+k], :]."""
    Yp = _f64(Y_perm)
    w = _f64(topk_w)
    T, K = w.shape
    rows = np.asarray(pair_to_row).astype(np.int64).reshape(T, K)
    Y = np.zeros((T, Yp.shape[1]), F64)
    for k in range(K):
        Y += w[:, k:k + 1] * Yp[rows[:, k]]
    return Y


# --------------------------------------------------------------------------------------------
# O5  unpermute-combine backward
# --------------------------------------------------------------------------------------------
def unpermute_combine_bwd(dY, Y_perm, topk_w, pair_to_row):
    """dYp[pair_to_row[p],:] = w(p) * dY[t(p),:];  dw[t,k] = <dY[t,:], Yp[pair_to_row[t*K+k],:]>."""
    dY = _f64(dY)
    Yp = _f64(Y_perm)
    w = _f64(topk_w)
    T, K = w.shape
    rows = np.asarray(pair_to_row).astype(np.int64).reshape(T, K)
    dYp = np.zeros((T * K, dY.shape[1]), F64)
    dw = np.zeros((T, K), F64)
    for k in range(K):
        dYp[rows[:, k]] = w[:, k:k + 1] * dY
        dw[:, k] = np.sum(dY * Yp[rows[:, k]], axis=1)
    return dYp, dw


# --------------------------------------------------------------------------------------------
# O6  down backward: dgrad + wgrad
# --------------------------------------------------------------------------------------------
def down_bwd(dY_perm, H_act, W_down, offsets):
    """dHact[r,:] = dYp[r,:] @ Wd[e]^T;  dWd[e] = Hact_e^T @ dYp_e  (zero for an empty expert)."""
    dYp = _f64(dY_perm)
    Hact = _f64(H_act)
    E, I, H = W_down.shape
    dHact = np.zeros((dYp.shape[0], I), F64)
    dWd = np.zeros((E, I, H), F64)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        dHact[r0:r1] = dYp[r0:r1] @ _f64(W_down[e]).T
        dWd[e] = Hact[r0:r1].T @ dYp[r0:r1]
    return dHact, dWd


# --------------------------------------------------------------------------------------------
# O7  SwiGLU backward + gate/up backward: dgrad + wgrad (the paper's dW1)
# --------------------------------------------------------------------------------------------
def swiglu_bwd(dH_act, GU):
    """dGU = [dg | du] with s = sigmoid(g): dg = dHact*u*s*(1+g*(1-s)), du = dHact*g*s."""
    dHact = _f64(dH_act)
    GU = _f64(GU)
    I = dHact.shape[1]
    g, u = GU[:, :I], GU[:, I:]
    s = 1.0 / (1.0 + np.exp(-g))
    dg = dHact * u * s * (1.0 + g * (1.0 - s))
    du = dHact * g * s
    return np.concatenate([dg, du], axis=1)


def down_dgrad_swiglu_bwd(dY_perm, W_down, GU, offsets):
    """The fused call's result: dGU = swiglu_bwd(dHact, GU) with dHact[r,:] = dYp[r,:] @ Wd[e]^T, the two
    definitions above applied one after the other with nothing rounded in between."""
    dYp = _f64(dY_perm)
    E, I, H = W_down.shape
    dHact = np.zeros((dYp.shape[0], I), F64)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 > r0:
            dHact[r0:r1] = dYp[r0:r1] @ _f64(W_down[e]).T
    return swiglu_bwd(dHact, GU)


def gateup_bwd_from_dgu(dGU, X_perm, W_gate, W_up, offsets):
    """dXp[r,:] = dg[r,:] @ Wg[e]^T + du[r,:] @ Wu[e]^T;  dWg[e] = Xp_e^T @ dg_e;  dWu likewise."""
    dGU = _f64(dGU)
    Xp = _f64(X_perm)
    E, H, I = W_gate.shape
    dXp = np.zeros((Xp.shape[0], H), F64)
    dWg = np.zeros((E, H, I), F64)
    dWu = np.zeros((E, H, I), F64)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        dg, du = dGU[r0:r1, :I], dGU[r0:r1, I:]
        dXp[r0:r1] = dg @ _f64(W_gate[e]).T + du @ _f64(W_up[e]).T
        dWg[e] = Xp[r0:r1].T @ dg
        dWu[e] = Xp[r0:r1].T @ du
    return dXp, dWg, dWu


def gateup_swiglu_bwd(dH_act, GU, X_perm, W_gate, W_up, offsets):
    """Returns dGU [R,2I], dXp [R,H], dWg, dWu [E,H,I]."""
    dGU = swiglu_bwd(dH_act, GU)
    dXp, dWg, dWu = gateup_bwd_from_dgu(dGU, X_perm, W_gate, W_up, offsets)
    return dGU, dXp, dWg, dWu


# --------------------------------------------------------------------------------------------
# O8  permute backward
# --------------------------------------------------------------------------------------------
def permute_bwd(dX_perm, pair_to_row, T, K):
    """dX[t,:] = sum_k dXp[pair_to_row[t*K+k], :]."""
    dXp = _f64(dX_perm)
    rows = np.asarray(pair_to_row).astype(np.int64).reshape(T, K)
    dX = np.zeros((T, dXp.shape[1]), F64)
    for k in range(K):
        dX += dXp[rows[:, k]]
    return dX


# --------------------------------------------------------------------------------------------
# The whole layer, chained in fp64 with no intermediate rounding ("exact" mode)
# --------------------------------------------------------------------------------------------
def layer_fwd(X, topk_idx, topk_w, W_gate, W_up, W_down):
    E = W_gate.shape[0]
    Xp, counts, offsets, row_to_pair, pair_to_row = permute(X, topk_idx, E)
    Hact, GU = gateup_swiglu(Xp, W_gate, W_up, offsets)
    Yp = down(Hact, W_down, offsets)
    Y = unpermute_combine(Yp, topk_w, pair_to_row)
    return dict(X_perm=Xp, counts=counts, offsets=offsets, row_to_pair=row_to_pair,
                pair_to_row=pair_to_row, H_act=Hact, GU=GU, Y_perm=Yp, Y=Y)


def layer_fwd_bwd(X, topk_idx, topk_w, W_gate, W_up, W_down, dY):
    """Forward then backward of L = sum(dY * Y) with the routing indices frozen."""
    f = layer_fwd(X, topk_idx, topk_w, W_gate, W_up, W_down)
    T, K = np.asarray(topk_idx).shape
    dYp, dw = unpermute_combine_bwd(dY, f["Y_perm"], topk_w, f["pair_to_row"])
    dHact, dWd = down_bwd(dYp, f["H_act"], W_down, f["offsets"])
    dGU, dXp, dWg, dWu = gateup_swiglu_bwd(dHact, f["GU"], f["X_perm"], W_gate, W_up, f["offsets"])
    dX = permute_bwd(dXp, f["pair_to_row"], T, K)
    f.update(dY_perm=dYp, dtopk_w=dw, dH_act=dHact, dW_down=dWd, dGU=dGU, dX_perm=dXp,
             dW_gate=dWg, dW_up=dWu, dX=dX)
    return f


# ---- router in front of the layer (the step before route-permute) ------------------------------
def router_topk(logits, K):
    """Top-k routing as the benchmark workloads describe it: softmax over the router logits, the K
    largest per token kept and renormalised to sum 1.

    logits [T,E] float32.  Selection is decided on the float32 values as given: the K largest per
    row in descending order, equal values ordered by lower expert id (the comparison of two float32
    numbers is exact in any precision).  Renormalising softmax(z) over the selected set cancels the
    full denominator, so  w_k = exp(z_k) / sum_{j selected} exp(z_j),  evaluated in fp64 with the
    row maximum subtracted.  Returns topk_idx [T,K] int32, topk_w [T,K] float64.  Logits must be finite."""
    z32 = np.asarray(logits, dtype=np.float32)
    T, E = z32.shape
    assert 1 <= K <= E
    z = z32.astype(F64)
    ids = np.broadcast_to(np.arange(E), (T, E))
    order = np.lexsort((ids, -z), axis=1)          # primary key: value descending; secondary: id ascending
    idx = order[:, :K]
    zs = np.take_along_axis(z, idx, axis=1)
    ex = np.exp(zs - zs[:, :1])
    return idx.astype(np.int32), ex / ex.sum(axis=1, keepdims=True)


def router_topk_bwd(topk_idx, topk_w, dtopk_w, E):
    """Gradient of the renormalised top-k weights with respect to the logits, selection frozen:
    dz[t, idx[t,k]] = w_k * (dw_k - sum_j w_j dw_j); zero for experts that were not selected."""
    idx = np.asarray(topk_idx).astype(np.int64)
    w, dw = _f64(topk_w), _f64(dtopk_w)
    T, K = idx.shape
    inner = (w * dw).sum(axis=1, keepdims=True)
    dz = np.zeros((T, E), dtype=F64)
    np.put_along_axis(dz, idx, w * (dw - inner), axis=1)
    return dz


# ---- block-scaled FP8 (MXFP8) operands for the grouped GEMMs --------------------------------------
# Format (the OCP Microscaling "MXFP8" format the Blackwell tensor cores consume with kind::mxf8f6f4):
#   * elements: FP8 E4M3 -- 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinities, S.1111.111 is NaN,
#     largest finite value 448 = 1.75 * 2^8, subnormals m * 2^-9;
#   * one shared scale per block of 32 consecutive elements ALONG THE CONTRACTION AXIS: E8M0, i.e. the power of
#     two 2^(s - 127) stored as the byte s in [0, 254];
#   * the scale of a block with largest magnitude a > 0 is 2^(floor(log2 a) - 8) (8 = exponent of the largest E4M3
#     power of two), clamped to the E8M0 range; the elements are v / scale rounded to nearest even onto the E4M3
#     grid, magnitudes above 448 saturating to 448; an all-zero block takes the smallest scale and zero codes.
# The paper itself only names FP8 tensor-core paths among its micro-profiling tools; this is the Blackwell follow-up
# of the bf16 GEMMs and is held to its own tolerance (a 3-bit mantissa cannot meet the bf16 bounds).
E4M3_MAX = 448.0
MX_BLOCK = 32


def e4m3_decode(codes):
    """uint8 E4M3 codes -> float64 values (NaN for the two NaN codes)."""
    c = np.asarray(codes).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(F64)
    val = np.where(e == 0, m * 2.0 ** -9, (1.0 + m / 8.0) * np.exp2((e - 7).astype(F64)))
    val = np.where((e == 15) & ((c & 0x7) == 7), np.nan, val)
    return sign * val


def e4m3_encode(y):
    """float64 -> uint8 E4M3 codes: round to nearest, ties to even, magnitudes above 448 saturate to 448."""
    y = _f64(y)
    a = np.minimum(np.abs(y), 1e30)
    # spacing of the E4M3 grid around a: 2^-9 below the smallest normal 2^-6, else 2^(floor(log2 a) - 3)
    ex = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))
    step = np.exp2(ex - 3.0)
    q = np.rint(a / step) * step            # numpy rint = round half to even; a/step is exact (step a power of two)
    q = np.minimum(q, E4M3_MAX)
    # q back to fields
    qe = np.floor(np.log2(np.maximum(q, 2.0 ** -6)))
    is_sub = q < 2.0 ** -6
    e_field = np.where(is_sub, 0, qe + 7).astype(np.int64)
    m_field = np.where(is_sub, np.rint(q * 2.0 ** 9), np.rint((q / np.exp2(qe) - 1.0) * 8.0)).astype(np.int64)
    code = (e_field << 3) | m_field
    code = np.where(np.signbit(y), code | 0x80, code)
    return code.astype(np.uint8)


def mxfp8_quantize(x):
    """Block-scaled FP8 quantisation along the LAST axis (length a multiple of 32).

    Returns (codes uint8 same shape, scales uint8 [..., n/32], dequantised float64 same shape)."""
    x = _f64(x)
    n = x.shape[-1]
    assert n % MX_BLOCK == 0
    blocks = x.reshape(x.shape[:-1] + (n // MX_BLOCK, MX_BLOCK))
    amax = np.max(np.abs(blocks), axis=-1)
    safe = np.where(amax > 0, amax, 1.0)
    s_exp = np.where(amax > 0, np.floor(np.log2(safe)) - 8.0, -127.0)
    s_exp = np.clip(s_exp, -127.0, 127.0)
    scale = np.exp2(s_exp)
    codes = e4m3_encode(blocks / scale[..., None])
    deq = e4m3_decode(codes) * scale[..., None]
    return codes.reshape(x.shape), (s_exp + 127.0).astype(np.uint8), deq.reshape(x.shape)


def down_mxfp8(H_act, W_down, offsets):
    """The down projection with both operands block-scaled FP8 along the contraction (I):
    Yp[r,:] = Q(Hact[r,:]) @ Q(Wd[e]) where Q quantises Hact row-wise in blocks of 32 along I and Wd[e] column-wise
    in blocks of 32 along I (each output feature h has its own scales), and the product of the dequantised
    operands is taken exactly.  Returns Yp [R,H] float64."""
    _, _, a_deq = mxfp8_quantize(H_act)
    Wt = np.swapaxes(_f64(W_down), 1, 2)                 # [E, H, I]: contraction last
    _, _, b_deq = mxfp8_quantize(Wt)
    return down(a_deq, np.swapaxes(b_deq, 1, 2), offsets)


def down_dgrad_mxfp8(dY_perm, W_down, offsets):
    """The data gradient of the down projection with both operands block-scaled FP8 along ITS contraction (H):
    dHact[r,:] = Q(dYp[r,:]) @ Q(Wd[e])^T where Q quantises dYp row-wise in blocks of 32 along H and Wd[e] [I,H]
    row-wise in blocks of 32 along H (each intermediate feature i has its own scales), and the product of the
    dequantised operands is taken exactly.  Returns dHact [R,I] float64."""
    _, _, a_deq = mxfp8_quantize(dY_perm)
    _, _, b_deq = mxfp8_quantize(_f64(W_down))           # [E, I, H]: contraction last as it lies
    E = b_deq.shape[0]
    out = np.zeros((a_deq.shape[0], b_deq.shape[1]), dtype=F64)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi > lo:
            out[lo:hi] = a_deq[lo:hi] @ b_deq[e].T
    return out


def gateup_dgrad_mxfp8(dGU, W_gate, W_up, offsets):
    """The data gradient of the gate/up projection with block-scaled FP8 operands along ITS contraction (the 2I gate
    and up features): dXp[r,:] = Q(dGU[r,:I]) @ Q(Wg[e])^T + Q(dGU[r,I:]) @ Q(Wu[e])^T, where Q quantises dGU row-wise in
    blocks of 32 along its 2I columns (I is a multiple of 32, so no block straddles the gate/up boundary) and Wg[e],
    Wu[e] [H,I] row-wise in blocks of 32 along I; the products of the dequantised operands are taken exactly.
    Returns dXp [R,H] float64."""
    I = W_gate.shape[2]
    assert I % MX_BLOCK == 0 and dGU.shape[1] == 2 * I
    _, _, a_deq = mxfp8_quantize(dGU)
    _, _, g_deq = mxfp8_quantize(_f64(W_gate))           # [E, H, I]: contraction last as it lies
    _, _, u_deq = mxfp8_quantize(_f64(W_up))
    out = np.zeros((a_deq.shape[0], W_gate.shape[1]), dtype=F64)
    for e in range(W_gate.shape[0]):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi > lo:
            out[lo:hi] = a_deq[lo:hi, :I] @ g_deq[e].T + a_deq[lo:hi, I:] @ u_deq[e].T
    return out


def gateup_mxfp8(X_perm, W_gate, W_up, offsets):
    """The gate/up projection with block-scaled FP8 operands along its contraction (H): g = Q(Xp[r,:]) @ Q(Wg[e]),
    u = Q(Xp[r,:]) @ Q(Wu[e]), where Q quantises Xp row-wise in blocks of 32 along H and each weight column
    Wg[e][:,i], Wu[e][:,i] in blocks of 32 along H (every gate / up feature has its own scales); the products of the
    dequantised operands are taken exactly.  Returns the pre-activations GU [R,2I] = [g | u] float64."""
    _, _, a_deq = mxfp8_quantize(X_perm)
    g_deq = np.swapaxes(mxfp8_quantize(np.swapaxes(_f64(W_gate), 1, 2))[2], 1, 2)      # quantised along H, back to [E,H,I]
    u_deq = np.swapaxes(mxfp8_quantize(np.swapaxes(_f64(W_up), 1, 2))[2], 1, 2)
    return gateup_swiglu(a_deq, g_deq, u_deq, offsets)[1]


def swiglu_fwd(GU):
    """Hact = silu(g) * u with [g | u] = GU, silu(g) = g / (1 + exp(-g)).  Returns Hact [R,I] float64."""
    GU = _f64(GU)
    I = GU.shape[1] // 2
    g, u = GU[:, :I], GU[:, I:]
    return g / (1.0 + np.exp(-g)) * u


def wgrad_mxfp8(A_rows, B_rows, offsets):
    """A weight gradient with block-scaled FP8 operands along ITS contraction, the packed rows of each expert:
    dW[e] = Q(A_e)^T @ Q(B_e) with A_e = A_rows[offsets[e]:offsets[e+1], :] ([n_e, M]) and B_e likewise ([n_e, N]), where Q
    quantises every COLUMN in blocks of 32 consecutive rows counted from the expert's first row (a block never holds
    rows of two experts; the expert's last block may be short and is scaled by the rows it has).  The product of the
    dequantised operands is taken exactly; an expert without rows gives zeros.  Returns dW [E, M, N] float64.
    (down projection: A = H_act, B = dY_perm; gate/up projection: A = X_perm, B = dGU, dW = [dW_gate | dW_up].)"""
    A, B = _f64(A_rows), _f64(B_rows)
    E = len(offsets) - 1
    out = np.zeros((E, A.shape[1], B.shape[1]), dtype=F64)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        n = hi - lo
        if n == 0:
            continue
        pad = (-n) % MX_BLOCK
        at = np.concatenate([A[lo:hi].T, np.zeros((A.shape[1], pad))], axis=1)       # [M, n + pad]: contraction last
        bt = np.concatenate([B[lo:hi].T, np.zeros((B.shape[1], pad))], axis=1)
        out[e] = mxfp8_quantize(at)[2] @ mxfp8_quantize(bt)[2].T
    return out
