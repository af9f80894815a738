"""Router entry points against the oracle: indices bit for bit (selection is decided on the float32
logits on both sides), weights and logit gradients in fp32 arithmetic against fp64.

Tolerances: a weight is exp(z_k - z_max) / sum over at most 32 terms, all in fp32 with expf (<= 2 ulp):
relative error below ~40 * 2^-24 = 2.4e-6; the test allows 1e-5 relative (+1e-7 absolute for weights that
underflow towards zero).  The gradient is a product / difference of such values: 1e-5 of the row maximum."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2606_26453_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_router(z32, K):
    from paper_2606_26453_b200 import binding as B
    T, E = z32.shape
    d = B.dims(T, 64, 64, E, K)
    z = torch.from_numpy(z32).cuda()
    idx = torch.empty((T, K), dtype=torch.int32, device="cuda")
    w = torch.empty((T, K), dtype=torch.float32, device="cuda")
    B.moe_router_topk(d, z, idx, w)
    torch.cuda.synchronize()
    return d, idx, w


def check_forward(z32, K):
    d, idx, w = run_router(z32, K)
    ridx, rw = O.router_topk(z32, K)
    assert np.array_equal(idx.cpu().numpy(), ridx)
    np.testing.assert_allclose(w.cpu().numpy().astype(np.float64), rw, rtol=1e-5, atol=1e-7)
    return d, idx, w, ridx, rw


CASES = [(256, 8, 2), (1000, 64, 6), (777, 128, 8), (130, 60, 5), (64, 1024, 32), (33, 1000, 7), (50, 5, 5), (19, 1, 1),
         (300, 33, 1)]


@pytest.mark.parametrize("T,E,K", CASES)
def test_router_forward_and_backward(T, E, K):
    from paper_2606_26453_b200 import binding as B
    rng = np.random.default_rng(T * 1000 + E)
    z32 = rng.standard_normal((T, E)).astype(np.float32)
    d, idx, w, ridx, rw = check_forward(z32, K)
    dw = rng.standard_normal((T, K)).astype(np.float32)
    dz = torch.full((T, E), 7.0, dtype=torch.float32, device="cuda")          # must be overwritten in full
    B.moe_router_topk_bwd(d, idx, w, torch.from_numpy(dw).cuda(), dz)
    torch.cuda.synchronize()
    ref = O.router_topk_bwd(ridx, rw, dw, E)                                   # the oracle's own weights
    got = dz.cpu().numpy().astype(np.float64)
    unselected = np.ones((T, E), dtype=bool)
    np.put_along_axis(unselected, ridx.astype(np.int64), False, axis=1)
    assert not got[unselected].any()                                           # exact zeros where nothing was kept
    np.testing.assert_allclose(got, ref, rtol=1e-5, atol=1e-5 * max(1e-30, np.abs(ref).max()))


def test_router_ties_and_extreme_logits():
    # exact ties everywhere: lower ids win, in id order; equal weights
    z = np.zeros((40, 96), dtype=np.float32)
    check_forward(z, 8)
    # few distinct values: many ties inside and at the edge of the kept set
    rng = np.random.default_rng(0)
    z = rng.integers(-2, 3, size=(500, 70)).astype(np.float32)
    check_forward(z, 9)
    # large spread: weights underflow to zero without NaN; -inf logits are never preferred over finite ones
    z = (rng.standard_normal((200, 40)) * 60).astype(np.float32)
    z[:, 7] = -np.inf
    d, idx, w, ridx, rw = check_forward(z, 4)
    assert torch.isfinite(w).all() and not bool((idx == 7).any())


@pytest.mark.parametrize("name", ["tiny", "fine_grained", "many_small", "few_large"])
def test_router_reproduces_the_workload_routing(name):
    """Full-size logits of the benchmark workloads: indices against the oracle bit for bit on every token, and
    against the routing the workload generator made from the same draw."""
    cfg = W.CONFIGS[name]
    z32 = W.make_router_logits(cfg)
    d, idx, w, ridx, rw = check_forward(z32, cfg.K)
    gen_idx, gen_w = W.make_routing(cfg)
    same = (idx.cpu().numpy() == gen_idx).all(axis=1)
    # the generator decides on float64 logits: a token can differ only where two of its float32 logits collide
    assert same.mean() > 0.999
    np.testing.assert_allclose(w.cpu().numpy()[same], gen_w[same], rtol=2.0 ** -7)


def test_router_feeds_the_layer():
    """Router -> permute: the routing the kernel produced drives a1 and gives the oracle's packed order."""
    from paper_2606_26453_b200 import binding as B
    cfg = W.CONFIGS["tiny"]
    z32 = W.make_router_logits(cfg)
    d, idx, w = run_router(z32, cfg.K)
    dl = B.dims(cfg.T, cfg.H, cfg.I, cfg.E, cfg.K)
    R = cfg.R
    i32 = lambda n: torch.empty(n, dtype=torch.int32, device="cuda")
    counts, offsets, r2p, p2r = i32(cfg.E), i32(cfg.E + 1), i32(R), i32(R)
    ws = torch.empty(B.moe_permute_workspace_bytes(dl), dtype=torch.uint8, device="cuda")
    B.moe_permute(dl, None, idx, None, counts, offsets, r2p, p2r, ws)
    torch.cuda.synchronize()
    rc, ro, rr, rp = O.permute_indices(O.router_topk(z32, cfg.K)[0], cfg.E)
    assert np.array_equal(counts.cpu().numpy(), rc) and np.array_equal(offsets.cpu().numpy(), ro)
    assert np.array_equal(r2p.cpu().numpy(), rr) and np.array_equal(p2r.cpu().numpy(), rp)
