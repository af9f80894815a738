"""Pins for the fp64 oracle: every check here compares the oracle with something that is not the
oracle (a brute-force loop, a library routine used in a different formulation, autograd, finite
differences, a closed form), chosen so that a dropped term, a wrong sign, a transposed operand or
a wrong index anywhere in oracle/moe_oracle.py fails at least one of them.  CPU only."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2606_26453_b200 import workloads as W

torch.set_default_dtype(torch.float64)


def small_problem(T=24, H=16, I=24, E=5, K=3, seed=0, empty=()):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((T, H))
    Wg = rng.standard_normal((E, H, I)) * 0.3
    Wu = rng.standard_normal((E, H, I)) * 0.3
    Wd = rng.standard_normal((E, I, H)) * 0.3
    dY = rng.standard_normal((T, H))
    z = rng.standard_normal((T, E))
    for e in empty:
        z[:, e] = -1e9
    idx = np.argsort(-z, axis=1, kind="stable")[:, :K].astype(np.int32)
    w = rng.dirichlet(np.ones(K), size=T)
    return X, idx, w, Wg, Wu, Wd, dY


# ------------------------------------------------------------------------------------------
# O1: permutation indices
# ------------------------------------------------------------------------------------------
def brute_force_permute(idx, E):
    """The counting-sort definition written as plain loops (pairs visited in ascending p)."""
    T, K = idx.shape
    R = T * K
    counts = [0] * E
    for t in range(T):
        for k in range(K):
            counts[idx[t, k]] += 1
    offsets = [0] * (E + 1)
    for e in range(E):
        offsets[e + 1] = offsets[e] + counts[e]
    cur = list(offsets[:E])
    row_to_pair = [-1] * R
    pair_to_row = [-1] * R
    for p in range(R):
        e = idx[p // K, p % K]
        r = cur[e]
        cur[e] += 1
        row_to_pair[r] = p
        pair_to_row[p] = r
    return counts, offsets, row_to_pair, pair_to_row


@pytest.mark.parametrize("T,E,K,seed", [(1, 1, 1, 0), (7, 3, 2, 1), (50, 9, 4, 2), (33, 16, 1, 3), (64, 4, 4, 4)])
def test_permute_indices_brute_force(T, E, K, seed):
    rng = np.random.default_rng(seed)
    idx = rng.integers(0, E, size=(T, K)).astype(np.int32)       # duplicates within a token allowed
    if E > 2:
        idx[idx == 1] = 0                                          # force an empty expert
    counts, offsets, r2p, p2r = O.permute_indices(idx, E)
    bc, bo, br2p, bp2r = brute_force_permute(idx, E)
    assert counts.tolist() == bc
    assert offsets.tolist() == bo
    assert r2p.tolist() == br2p
    assert p2r.tolist() == bp2r
    assert counts.dtype == offsets.dtype == r2p.dtype == p2r.dtype == np.int32


def test_permute_indices_library_stable_sort_and_invariants():
    cfg = W.CONFIGS["tiny"]
    idx, _ = W.make_routing(cfg)
    counts, offsets, r2p, p2r = O.permute_indices(idx, cfg.E)
    flat = torch.from_numpy(idx.reshape(-1).astype(np.int64))
    sorted_e, order = torch.sort(flat, stable=True)
    assert np.array_equal(order.numpy(), r2p)
    R = cfg.R
    assert counts.sum() == R and offsets[0] == 0 and offsets[-1] == R
    assert np.all(np.diff(offsets) == counts)
    assert np.array_equal(np.sort(r2p), np.arange(R))
    assert np.array_equal(p2r[r2p], np.arange(R))
    e_of_row = idx.reshape(-1)[r2p]
    assert np.all(np.diff(e_of_row) >= 0)
    for e in range(cfg.E):
        seg = r2p[offsets[e]:offsets[e + 1]]
        assert np.all(np.diff(seg) > 0)                            # stable: p ascending inside an expert
        assert np.all(e_of_row[offsets[e]:offsets[e + 1]] == e)
    assert np.all(np.bincount(r2p // cfg.K, minlength=cfg.T) == cfg.K)


def test_offsets_are_the_shifted_inclusive_cumsum():
    """The paper's kernel indexes experts with an inclusive cumulative sum of row counts:
    start = (e ? cumsum[e-1] : 0), end = cumsum[e].  offsets[1:] must be that vector."""
    idx = np.array([[2, 0], [2, 2], [3, 0]], dtype=np.int32)
    counts, offsets, _, _ = O.permute_indices(idx, 5)
    inclusive = np.cumsum([2, 0, 3, 1, 0])
    assert counts.tolist() == [2, 0, 3, 1, 0]
    assert offsets[1:].tolist() == inclusive.tolist()
    for e in range(5):
        start = inclusive[e - 1] if e else 0
        assert (offsets[e], offsets[e + 1]) == (start, inclusive[e])


def test_permute_rows_are_copies():
    X, idx, *_ = small_problem()
    Xp, counts, offsets, r2p, p2r = O.permute(X, idx, 5)
    K = idx.shape[1]
    for r in range(Xp.shape[0]):
        assert np.array_equal(Xp[r], X[r2p[r] // K])


# ------------------------------------------------------------------------------------------
# forward: dense special cases, per-token loop
# ------------------------------------------------------------------------------------------
def dense_mlp_torch(X, Wg, Wu, Wd):
    X, Wg, Wu, Wd = map(torch.from_numpy, (X, Wg, Wu, Wd))
    return (torch.nn.functional.silu(X @ Wg) * (X @ Wu)) @ Wd


def test_single_expert_top1_is_dense_swiglu_mlp():
    rng = np.random.default_rng(5)
    T, H, I = 19, 12, 20
    X = rng.standard_normal((T, H))
    Wg, Wu = rng.standard_normal((1, H, I)), rng.standard_normal((1, H, I))
    Wd = rng.standard_normal((1, I, H))
    idx = np.zeros((T, 1), np.int32)
    w = np.ones((T, 1))
    f = O.layer_fwd(X, idx, w, Wg, Wu, Wd)
    ref = dense_mlp_torch(X, Wg[0], Wu[0], Wd[0]).numpy()
    np.testing.assert_allclose(f["Y"], ref, rtol=1e-12, atol=1e-12)
    # non-square shapes make a transposed operand a shape error; also check GU halves separately
    np.testing.assert_allclose(f["GU"][:, :I], X @ Wg[0], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(f["GU"][:, I:], X @ Wu[0], rtol=1e-12, atol=1e-12)


def test_identical_experts_equal_dense_mlp_for_any_routing():
    X, idx, w, Wg, Wu, Wd, _ = small_problem(seed=3)
    Wg[:] = Wg[0]
    Wu[:] = Wu[0]
    Wd[:] = Wd[0]
    f = O.layer_fwd(X, idx, w, Wg, Wu, Wd)          # Dirichlet weights sum to one
    ref = dense_mlp_torch(X, Wg[0], Wu[0], Wd[0]).numpy()
    np.testing.assert_allclose(f["Y"], ref, rtol=1e-11, atol=1e-11)


def per_token_forward(X, idx, w, Wg, Wu, Wd):
    T, H = X.shape
    K = idx.shape[1]
    I = Wg.shape[2]
    Y = np.zeros((T, H))
    for t in range(T):
        for k in range(K):
            e = idx[t, k]
            g = np.array([np.dot(X[t], Wg[e][:, i]) for i in range(I)])
            u = np.array([np.dot(X[t], Wu[e][:, i]) for i in range(I)])
            h = g * (1.0 / (1.0 + np.exp(-g))) * u
            y = np.array([np.dot(h, Wd[e][:, j]) for j in range(H)])
            Y[t] += w[t, k] * y
    return Y


@pytest.mark.parametrize("empty", [(), (0,), (4,), (1, 2)])
def test_per_token_loop(empty):
    X, idx, w, Wg, Wu, Wd, _ = small_problem(T=13, H=8, I=10, E=5, K=2, seed=7, empty=empty)
    f = O.layer_fwd(X, idx, w, Wg, Wu, Wd)
    np.testing.assert_allclose(f["Y"], per_token_forward(X, idx, w, Wg, Wu, Wd), rtol=1e-12, atol=1e-12)
    for e in empty:
        assert f["counts"][e] == 0


def test_forward_linear_in_routing_weights_and_token_equivariant():
    X, idx, w, Wg, Wu, Wd, _ = small_problem(seed=11)
    f1 = O.layer_fwd(X, idx, w, Wg, Wu, Wd)["Y"]
    f2 = O.layer_fwd(X, idx, 2.5 * w, Wg, Wu, Wd)["Y"]
    np.testing.assert_allclose(f2, 2.5 * f1, rtol=1e-12, atol=1e-12)
    perm = np.random.default_rng(0).permutation(X.shape[0])
    f3 = O.layer_fwd(X[perm], idx[perm], w[perm], Wg, Wu, Wd)["Y"]
    np.testing.assert_allclose(f3, f1[perm], rtol=1e-12, atol=1e-12)


def test_silu_closed_forms():
    g = np.array([[0.0, 1.0, -1.0, 30.0, -30.0]])
    u = np.ones_like(g)
    dGU = O.swiglu_bwd(np.ones_like(g), np.concatenate([g, u], axis=1))
    s1 = 1 / (1 + np.exp(-1.0))
    np.testing.assert_allclose(dGU[0, 0], 0.5)                                     # silu'(0) = 1/2
    np.testing.assert_allclose(dGU[0, 1], s1 * (1 + 1 * (1 - s1)))
    np.testing.assert_allclose(dGU[0, 3], 1.0, atol=1e-10)                         # silu ~ identity
    np.testing.assert_allclose(dGU[0, 4], 0.0, atol=1e-10)
    np.testing.assert_allclose(dGU[0, 5:], g[0] / (1 + np.exp(-g[0])))           # du = silu(g)
    Xp = np.eye(5)[:1]
    Hact, GU = O.gateup_swiglu(Xp, g.reshape(1, 1, 5).repeat(5, 1), np.ones((1, 5, 5)), [0, 1])
    np.testing.assert_allclose(Hact[0], g[0] / (1 + np.exp(-g[0])))


# ------------------------------------------------------------------------------------------
# A18: permute / unpermute identities
# ------------------------------------------------------------------------------------------
def test_permute_unpermute_identities():
    rng = np.random.default_rng(2)
    T, H, E = 40, 8, 6
    X = rng.standard_normal((T, H))
    idx1 = rng.integers(0, E, size=(T, 1)).astype(np.int32)
    Xp, _, _, _, p2r = O.permute(X, idx1, E)
    assert np.array_equal(O.unpermute_combine(Xp, np.ones((T, 1)), p2r), X)      # K=1: identity
    assert np.array_equal(O.permute_bwd(Xp, p2r, T, 1), X)
    K = 4
    idx = np.argsort(rng.standard_normal((T, E)), axis=1)[:, :K].astype(np.int32)
    Xp, _, _, _, p2r = O.permute(X, idx, E)
    np.testing.assert_allclose(O.unpermute_combine(Xp, np.ones((T, K)), p2r), K * X, rtol=1e-15)
    assert np.array_equal(O.unpermute_combine(Xp, np.full((T, K), 0.25), p2r), X)  # power of two: exact
    np.testing.assert_allclose(O.permute_bwd(Xp, p2r, T, K), K * X, rtol=1e-15)


# ------------------------------------------------------------------------------------------
# backward: autograd on an independent formulation, finite differences, empty experts
# ------------------------------------------------------------------------------------------
def torch_per_token_loss(X, idx, w, Wg, Wu, Wd, dY):
    T, K = idx.shape
    Y = []
    for t in range(T):
        y = 0
        for k in range(K):
            e = int(idx[t, k])
            h = torch.nn.functional.silu(X[t] @ Wg[e]) * (X[t] @ Wu[e])
            y = y + w[t, k] * (h @ Wd[e])
        Y.append(y)
    Y = torch.stack(Y)
    return (Y * dY).sum()


@pytest.mark.parametrize("empty", [(), (0, 3)])
def test_backward_matches_autograd_per_token(empty):
    Xn, idx, wn, Wgn, Wun, Wdn, dYn = small_problem(T=11, H=6, I=9, E=5, K=2, seed=21, empty=empty)
    f = O.layer_fwd_bwd(Xn, idx, wn, Wgn, Wun, Wdn, dYn)
    X, w, Wg, Wu, Wd = (torch.tensor(a, requires_grad=True) for a in (Xn, wn, Wgn, Wun, Wdn))
    torch_per_token_loss(X, idx, w, Wg, Wu, Wd, torch.from_numpy(dYn)).backward()
    for name, ref in (("dX", X.grad), ("dtopk_w", w.grad), ("dW_gate", Wg.grad), ("dW_up", Wu.grad),
                      ("dW_down", Wd.grad)):
        np.testing.assert_allclose(f[name], ref.numpy(), rtol=1e-10, atol=1e-11, err_msg=name)
    for e in empty:
        assert not f["dW_gate"][e].any() and not f["dW_up"][e].any() and not f["dW_down"][e].any()


def test_packed_intermediate_gradients_match_autograd():
    """Pins the per-call backward functions (their packed-layout intermediates) one by one."""
    Xn, idx, wn, Wgn, Wun, Wdn, dYn = small_problem(T=14, H=6, I=10, E=4, K=3, seed=33)
    f = O.layer_fwd_bwd(Xn, idx, wn, Wgn, Wun, Wdn, dYn)
    E, K, T = 4, 3, 14
    off, r2p, p2r = f["offsets"], f["row_to_pair"].astype(np.int64), f["pair_to_row"].astype(np.int64)
    X = torch.tensor(Xn)
    Xp = X[torch.from_numpy(r2p // K)].clone().requires_grad_(True)
    Wg, Wu, Wd = (torch.tensor(a) for a in (Wgn, Wun, Wdn))
    GU = torch.cat([torch.cat([Xp[off[e]:off[e + 1]] @ Wg[e], Xp[off[e]:off[e + 1]] @ Wu[e]], dim=1)
                    for e in range(E)]).clone()
    GU.retain_grad()
    I = Wgn.shape[2]
    Hact = torch.nn.functional.silu(GU[:, :I]) * GU[:, I:]
    Hact.retain_grad()
    Yp = torch.cat([Hact[off[e]:off[e + 1]] @ Wd[e] for e in range(E)])
    Yp.retain_grad()
    Y = (torch.tensor(wn).unsqueeze(-1) * Yp[torch.from_numpy(p2r).reshape(T, K)]).sum(1)
    (Y * torch.from_numpy(dYn)).sum().backward()
    for name, ref in (("dY_perm", Yp.grad), ("dH_act", Hact.grad), ("dGU", GU.grad), ("dX_perm", Xp.grad)):
        np.testing.assert_allclose(f[name], ref.numpy(), rtol=1e-10, atol=1e-11, err_msg=name)
    np.testing.assert_allclose(f["Y"], Y.detach().numpy(), rtol=1e-12, atol=1e-12)


def test_fused_down_dgrad_swiglu_bwd_is_the_gradient_of_the_loss_wrt_the_pre_activations():
    """The fused call's oracle: dGU from dY_perm, W_down and the saved pre-activations alone.  Pinned by torch
    autograd of sum(dY_perm * (silu(g) * u) @ Wd[e]) with respect to [g | u] (an expert without rows included), and
    by a central difference along a random direction."""
    Xn, idx, wn, Wgn, Wun, Wdn, dYn = small_problem(T=15, H=6, I=10, E=5, K=2, seed=41, empty=(3,))
    f = O.layer_fwd_bwd(Xn, idx, wn, Wgn, Wun, Wdn, dYn)
    off, I = f["offsets"], Wgn.shape[2]
    assert off[4] == off[3]                                   # the expert without rows is really there
    got = O.down_dgrad_swiglu_bwd(f["dY_perm"], Wdn, f["GU"], off)
    GU = torch.tensor(f["GU"]).requires_grad_(True)
    Wd, dYp = torch.tensor(Wdn), torch.tensor(f["dY_perm"])

    def loss(gu):
        h = torch.nn.functional.silu(gu[:, :I]) * gu[:, I:]
        return sum(((h[off[e]:off[e + 1]] @ Wd[e]) * dYp[off[e]:off[e + 1]]).sum() for e in range(Wd.shape[0]))

    loss(GU).backward()
    np.testing.assert_allclose(got, GU.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(got, f["dGU"], rtol=1e-12, atol=1e-13)      # and it is the chain's dGU
    rng = np.random.default_rng(5)
    D = rng.standard_normal(f["GU"].shape)
    eps = 1e-6
    with torch.no_grad():
        fd = (loss(torch.tensor(f["GU"] + eps * D)) - loss(torch.tensor(f["GU"] - eps * D))).item() / (2 * eps)
    assert abs(fd - float((got * D).sum())) <= 1e-7 * max(1.0, abs(fd))


def test_backward_central_differences():
    X, idx, w, Wg, Wu, Wd, dY = small_problem(T=10, H=7, I=9, E=4, K=2, seed=41)
    f = O.layer_fwd_bwd(X, idx, w, Wg, Wu, Wd, dY)
    args = dict(X=X, w=w, Wg=Wg, Wu=Wu, Wd=Wd)
    grads = dict(X=f["dX"], w=f["dtopk_w"], Wg=f["dW_gate"], Wu=f["dW_up"], Wd=f["dW_down"])

    def loss(a):
        return float(np.sum(dY * O.layer_fwd(a["X"], idx, a["w"], a["Wg"], a["Wu"], a["Wd"])["Y"]))

    rng = np.random.default_rng(0)
    for name in args:
        for _ in range(3):
            d = rng.standard_normal(args[name].shape)
            eps = 1e-6
            ap = dict(args); ap[name] = args[name] + eps * d
            am = dict(args); am[name] = args[name] - eps * d
            fd = (loss(ap) - loss(am)) / (2 * eps)
            an = float(np.sum(grads[name] * d))
            assert abs(fd - an) <= 1e-7 * max(1.0, abs(an)), (name, fd, an)
        # a few single coordinates
        flat = args[name].reshape(-1)
        for j in rng.integers(0, flat.size, size=3):
            d = np.zeros(flat.size); d[j] = 1.0; d = d.reshape(args[name].shape)
            eps = 1e-6
            ap = dict(args); ap[name] = args[name] + eps * d
            am = dict(args); am[name] = args[name] - eps * d
            fd = (loss(ap) - loss(am)) / (2 * eps)
            an = float(grads[name].reshape(-1)[j])
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, j, fd, an)


def test_identical_experts_backward_equals_dense():
    Xn, idx, wn, Wgn, Wun, Wdn, dYn = small_problem(seed=9)
    Wgn[:] = Wgn[0]; Wun[:] = Wun[0]; Wdn[:] = Wdn[0]
    f = O.layer_fwd_bwd(Xn, idx, wn, Wgn, Wun, Wdn, dYn)
    X, Wg, Wu, Wd = (torch.tensor(a, requires_grad=True) for a in (Xn, Wgn[0], Wun[0], Wdn[0]))
    Y = (torch.nn.functional.silu(X @ Wg) * (X @ Wu)) @ Wd
    (Y * torch.from_numpy(dYn)).sum().backward()
    np.testing.assert_allclose(f["dX"], X.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(f["dW_gate"].sum(0), Wg.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(f["dW_up"].sum(0), Wu.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(f["dW_down"].sum(0), Wd.grad.numpy(), rtol=1e-10, atol=1e-11)


def test_wgrad_is_xt_g_per_expert_on_a_heavy_tailed_load():
    """dW1_e = X_e^T G_e over ragged row counts drawn like the paper's routing model
    (Dirichlet(alpha=0.24)-multinomial, several empty experts), at a reduced size."""
    E, K = 32, 4
    counts = W.dirichlet_multinomial_counts(E, R=400, alpha=0.24, seed=1)
    assert (counts == 0).sum() >= 1
    rng = np.random.default_rng(3)
    H, I = 6, 5
    R = int(counts.sum())
    offsets = np.concatenate([[0], np.cumsum(counts)])
    Xp = rng.standard_normal((R, H))
    dGU = rng.standard_normal((R, 2 * I))
    Wg = rng.standard_normal((E, H, I)); Wu = rng.standard_normal((E, H, I))
    _, dWg, dWu = O.gateup_bwd_from_dgu(dGU, Xp, Wg, Wu, offsets)
    e_of_row = np.repeat(np.arange(E), counts)
    onehot = (e_of_row[:, None] == np.arange(E)[None, :]).astype(np.float64)
    ref = np.einsum("re,rh,rn->ehn", onehot, Xp, dGU)
    np.testing.assert_allclose(dWg, ref[:, :, :I], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dWu, ref[:, :, I:], rtol=1e-12, atol=1e-12)
    for e in np.flatnonzero(counts == 0):
        assert not dWg[e].any() and not dWu[e].any()


def test_down_bwd_einsum():
    rng = np.random.default_rng(8)
    counts = np.array([3, 0, 5, 1])
    offsets = np.concatenate([[0], np.cumsum(counts)])
    R, I, H, E = 9, 4, 6, 4
    dYp, Hact, Wd = rng.standard_normal((R, H)), rng.standard_normal((R, I)), rng.standard_normal((E, I, H))
    dHact, dWd = O.down_bwd(dYp, Hact, Wd, offsets)
    e_of_row = np.repeat(np.arange(E), counts)
    np.testing.assert_allclose(dHact, np.einsum("rh,rih->ri", dYp, Wd[e_of_row]), rtol=1e-12, atol=1e-12)
    onehot = (e_of_row[:, None] == np.arange(E)[None, :]).astype(np.float64)
    np.testing.assert_allclose(dWd, np.einsum("re,ri,rh->eih", onehot, Hact, dYp), rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------------------------------
# router (softmax, top-k, renormalise) and its backward
# ------------------------------------------------------------------------------------------
def _router_loop(z32, K):
    """Per-row selection by repeated arg-max with the tie rule, weights by the textbook formula."""
    T, E = z32.shape
    idx = np.zeros((T, K), dtype=np.int32)
    w = np.zeros((T, K))
    for t in range(T):
        taken = set()
        for k in range(K):
            best = None
            for e in range(E):
                if e in taken:
                    continue
                if best is None or z32[t, e] > z32[t, best]:
                    best = e
            taken.add(best)
            idx[t, k] = best
        p = np.exp(z32[t].astype(np.float64))
        p /= p.sum()                                  # full softmax ...
        w[t] = p[idx[t]] / p[idx[t]].sum()            # ... renormalised over the kept experts
    return idx, w


@pytest.mark.parametrize("T,E,K,seed", [(17, 8, 2, 0), (9, 33, 5, 1), (5, 4, 4, 2), (11, 64, 1, 3)])
def test_router_matches_selection_loop(T, E, K, seed):
    z = np.random.default_rng(seed).standard_normal((T, E)).astype(np.float32)
    z[0, :] = np.round(z[0, :])                        # a row with many exact ties
    idx, w = O.router_topk(z, K)
    ridx, rw = _router_loop(z, K)
    assert np.array_equal(idx, ridx)
    np.testing.assert_allclose(w, rw, rtol=1e-12, atol=0)
    np.testing.assert_allclose(w.sum(axis=1), 1.0, rtol=1e-14)


def test_router_full_k_is_library_softmax_and_ties_closed_form():
    from scipy.special import softmax
    z = np.random.default_rng(4).standard_normal((13, 12)).astype(np.float32)
    idx, w = O.router_topk(z, 12)
    full = softmax(z.astype(np.float64), axis=1)
    np.testing.assert_allclose(w, np.take_along_axis(full, idx.astype(np.int64), axis=1), rtol=1e-12)
    assert np.all(np.diff(np.take_along_axis(z, idx.astype(np.int64), axis=1), axis=1) <= 0)
    # all logits equal: the first K experts in id order, equal weights
    idx, w = O.router_topk(np.full((3, 10), 0.25, dtype=np.float32), 4)
    assert np.array_equal(idx, np.tile(np.arange(4, dtype=np.int32), (3, 1)))
    np.testing.assert_allclose(w, 0.25, rtol=1e-15)


def test_router_shift_invariance_and_generator_agreement():
    rng = np.random.default_rng(5)
    z = rng.integers(-8, 9, size=(20, 16)).astype(np.float32)       # shifts stay exact in float32
    i0, w0 = O.router_topk(z, 3)
    i1, w1 = O.router_topk(z + np.float32(5.0), 3)
    assert np.array_equal(i0, i1)
    np.testing.assert_allclose(w0, w1, rtol=1e-12)
    # the workload generator's own routing (written separately) from the same logits
    cfg = W.CONFIGS["tiny"]
    gen_idx, gen_w = W.make_routing(cfg)
    idx, w = O.router_topk(W.make_router_logits(cfg), cfg.K)
    assert np.array_equal(idx, gen_idx)
    np.testing.assert_allclose(w, gen_w, rtol=2.0 ** -8)          # the generator rounds its weights to bf16


def test_router_bwd_matches_finite_differences():
    rng = np.random.default_rng(6)
    T, E, K = 6, 9, 4
    z = rng.standard_normal((T, E)).astype(np.float32)
    c = rng.standard_normal((T, K))
    idx, w = O.router_topk(z, K)
    dz = O.router_topk_bwd(idx, w, c, E)

    def f(zz):                                       # selection frozen: weights of the same experts
        zs = np.take_along_axis(zz, idx.astype(np.int64), axis=1)
        ex = np.exp(zs - zs.max(axis=1, keepdims=True))
        return float((c * ex / ex.sum(axis=1, keepdims=True)).sum())

    z64 = z.astype(np.float64)
    num = np.zeros_like(z64)
    h = 1e-6
    for t in range(T):
        for e in range(E):
            zp, zm = z64.copy(), z64.copy()
            zp[t, e] += h
            zm[t, e] -= h
            num[t, e] = (f(zp) - f(zm)) / (2 * h)
    np.testing.assert_allclose(dz, num, rtol=1e-6, atol=1e-9)
    np.testing.assert_allclose(dz.sum(axis=1), 0.0, atol=1e-14)
    unselected = np.ones((T, E), dtype=bool)
    np.put_along_axis(unselected, idx.astype(np.int64), False, axis=1)
    assert np.all(dz[unselected] == 0.0)
