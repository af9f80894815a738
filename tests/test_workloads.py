"""Host-side checks of the seeded input generators (no GPU)."""
import math
import os

import numpy as np
import pytest

from paper_2606_26453_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_dw1_workload.txt")


def read_golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = (s.strip() for s in line.split("=", 1))
            out[k] = v
    return out


def test_round_to_bf16_is_rne():
    import torch
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 3
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]     # exact ties -> even
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(W.round_to_bf16(x), ref)


@pytest.mark.parametrize("name", ["tiny", "fine_grained"])
def test_routing_shapes_and_weights(name):
    cfg = W.CONFIGS[name]
    idx, w = W.make_routing(cfg)
    assert idx.shape == (cfg.T, cfg.K) and idx.dtype == np.int32
    assert idx.min() >= 0 and idx.max() < cfg.E
    assert all(len(set(r)) == cfg.K for r in idx[:64].tolist())      # distinct experts per token
    assert np.all(np.abs(w.sum(1) - 1) < 0.02)
    assert np.all(np.diff(w, axis=1) <= 0)                             # slots in descending logit order
    assert np.array_equal(w, W.round_to_bf16(w))
    idx2, w2 = W.make_routing(cfg)
    assert np.array_equal(idx, idx2) and np.array_equal(w, w2)        # seeded


def test_zipf_routing_has_the_requested_empty_experts():
    cfg = W.MoeConfig("z", T=2048, H=128, I=128, E=64, K=8, routing="zipf", n_empty=4, cfg_id=5)
    idx, w = W.make_routing(cfg)
    counts = np.bincount(idx.reshape(-1), minlength=cfg.E)
    assert (counts == 0).sum() == 4
    assert counts.max() > 8 * np.median(counts[counts > 0]) / 4
    assert all(len(set(r)) == cfg.K for r in idx[:64].tolist())


def test_routing_from_counts():
    counts = [0, 1, 127, 129, 0, 0, 255, 0]
    idx, w = W.make_routing_from_counts(counts, K=2)
    assert np.bincount(idx.reshape(-1), minlength=8).tolist() == counts


def test_load_generator_closed_forms():
    g = read_golden()
    E, R, alpha = int(g["E"]), int(g["R"]), float(g["dirichlet_alpha"])
    # uniform split: multinomial with equal p has CV ~ sqrt((E-1)/R)
    rng = np.random.default_rng(0)
    cvs = []
    for _ in range(200):
        c = rng.multinomial(R, np.full(E, 1 / E))
        cvs.append(c.std() / c.mean())
    assert abs(np.mean(cvs) - math.sqrt((E - 1) / R)) < 0.003
    # Dirichlet-multinomial: CV ~ sqrt((E-1)/(E*alpha+1)) ~ 2.0, the paper measured 2.13
    cvs, empties = [], []
    for s in range(100):
        c = W.dirichlet_multinomial_counts(E, R, alpha, seed=s)
        assert c.sum() == R
        cvs.append(c.std() / c.mean()); empties.append((c == 0).sum())
    assert abs(np.mean(cvs) - math.sqrt((E - 1) / (E * alpha + 1))) < 0.15
    assert abs(np.mean(cvs) - float(g["cv_measured"])) < 0.35
    assert np.mean(empties) > 5
    # algorithmic work of one dW1 call: 2*R*M*N
    assert abs(2 * R * int(g["M"]) * int(g["N"]) / 1e12 - 1.917) < 1e-3


def test_flop_accounting():
    cfg = W.CONFIGS["few_large"]
    assert cfg.R == 16384
    assert abs(cfg.flops_fwd_bwd / 1e12 - 17.3173) < 1e-3


def test_paper_workload_routing_matches_its_load_model():
    g = read_golden()
    cfg = W.CONFIGS["paper_dw1"]
    assert (cfg.H, 2 * cfg.I, cfg.E, cfg.K, cfg.R) == (int(g["M"]), int(g["N"]), int(g["E"]), int(g["top_k"]), int(g["R"]))
    idx, w = W.make_routing(cfg)
    counts = np.bincount(idx.reshape(-1), minlength=cfg.E)
    assert counts.sum() == cfg.R and (counts == 0).sum() >= 3
    cv = counts.std() / counts.mean()
    assert 1.3 < cv < 3.0                                  # heavy tail like the paper's measured 2.13
    assert abs(4.0 * cfg.R * cfg.H * cfg.I / 1e12 - 1.917) < 1e-3   # the dW1 call: 2*R*M*N
