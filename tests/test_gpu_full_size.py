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


def test_sampled_tokens_against_exact_chain(full):
    cfg, dev, b = full
    n_tok = {"few_large": 12, "paper_dw1": 8}.get(cfg.name, 24)
    rng = np.random.default_rng(cfg.cfg_id)
    toks = np.sort(rng.choice(cfg.T, size=n_tok, replace=False))
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


def test_sampled_weight_gradient_blocks_against_exact_chain(full):
    cfg, dev, b = full
    counts = b.counts.cpu().numpy()
    offsets = b.offsets.cpu().numpy()
    nonempty = np.flatnonzero(counts > 0)
    chosen = {int(nonempty[np.argmax(counts[nonempty])]), int(nonempty[np.argmin(counts[nonempty])]),
              int(nonempty[len(nonempty) // 2])}
    if cfg.name == "few_large":
        chosen = {int(nonempty[0])}
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
