"""Seeded random shapes and expert loads through the whole layer, against the fp64 oracle.

The fixed parity cases pin the tile edges one knows about; these draw dimensions (multiples of 64), expert counts,
top-k and per-expert row counts (with empty experts, single rows, tile-boundary sizes and one large expert mixed in)
so that every launch-shape decision of the library -- single-CTA tiles, CTA pairs, half-height last tiles, swapped
operand roles, weight-gradient pairs -- is crossed at sizes nobody picked by hand."""
import numpy as np
import pytest

from oracle import moe_oracle as O
from tests import helpers as Hh

pytestmark = pytest.mark.gpu

FLOAT_OUTPUTS = [("y", "Y"), ("dx", "dX"), ("dw_gate", "dW_gate"), ("dw_up", "dW_up"), ("dw_down", "dW_down"),
                 ("h_act", "H_act"), ("gu", "GU"), ("y_perm", "Y_perm"), ("dy_perm", "dY_perm"), ("dh_act", "dH_act"),
                 ("dgu", "dGU"), ("dx_perm", "dX_perm")]


def draw_case(seed):
    rng = np.random.default_rng(1000 + seed)
    H = 64 * int(rng.integers(1, 7))
    I = 64 * int(rng.integers(1, 7))
    E = int(rng.integers(1, 25))
    K = int(rng.integers(1, min(E, 6) + 1))
    # rows per expert: a level that decides the launch shapes (tens, a few hundred, several hundred) times a spread
    level = [20, 150, 330, 420, 600, 900][seed % 6]
    counts = np.maximum(0, rng.normal(level, 0.35 * level, size=E)).astype(np.int64)
    special = [0, 1, 127, 128, 129, 255, 256, 257, 384, 385, 511, 512, 513]
    for e in rng.choice(E, size=min(E, 3), replace=False):
        counts[e] = special[int(rng.integers(0, len(special)))]
    if E > 2 and seed % 3 == 0:
        counts[int(rng.integers(0, E))] = int(rng.integers(1200, 2200))       # one expert of many row tiles
    if int(counts.sum()) == 0:
        counts[0] = K
    # routable: the sum a multiple of K, and no expert with more rows than there are tokens
    for _ in range(64):
        counts[int(np.argmin(counts))] += (-int(counts.sum())) % K
        T = int(counts.sum()) // K
        if int(counts.max()) <= T:
            break
        counts[int(np.argmax(counts))] = T
    return counts, K, H, I


@pytest.mark.parametrize("seed", list(range(48)))
def test_random_layer_against_oracle(seed):
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    counts, K, H, I = draw_case(seed)
    if int(counts.sum()) % K or int(counts.max()) > int(counts.sum()) // K:
        pytest.skip("drawn counts cannot be routed without repeating an expert in a token")
    cfg, host = Hh.ragged_workload(list(counts), K=K, H=H, I=I, seed=100 + seed)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"],
                          host["dY"])
    b = Hh.run_cuda_layer(Hh.device_workload(host), cfg.E)
    for name in ("counts", "offsets", "row_to_pair", "pair_to_row"):
        assert np.array_equal(getattr(b, name).cpu().numpy(), ref[name]), (name, list(counts), K, H, I)
    for attr, key in FLOAT_OUTPUTS:
        Hh.assert_close(Hh.to_np64(getattr(b, attr)), ref[key], f"{key} counts={list(counts)} K={K} H={H} I={I}")
    Hh.assert_close(b.dtopk_w.cpu().numpy().astype(np.float64), ref["dtopk_w"], "dtopk_w")
    # the same layer with the down dgrad and the SwiGLU backward as the one fused call
    bf = Hh.run_cuda_layer(Hh.device_workload(host), cfg.E, fused_swiglu_bwd=True)
    for attr, key in FLOAT_OUTPUTS:
        if attr != "dh_act":                                  # never written by the fused chain
            Hh.assert_close(Hh.to_np64(getattr(bf, attr)), ref[key], f"fused chain {key} counts={list(counts)} K={K} H={H} I={I}")


@pytest.mark.parametrize("H,I,counts,K", [
    (1408, 2880, [300, 1, 129, 430, 0], 2),          # the real widths: 1408 = 5.5 x 256, 2880 = 45 x 64 (partial column tiles)
    (2880, 1408, [40, 700, 1, 0, 259], 1),
    (2880, 2880, [520, 528, 8], 2),               # rows per expert above the pair / fixed-tile thresholds
    (1408, 1408, [255, 257, 0, 600, 88], 2),
])
def test_real_widths_at_small_row_counts(H, I, counts, K):
    from paper_2606_26453_b200 import binding as B
    B.load_library()
    cfg, host = Hh.ragged_workload(counts, K=K, H=H, I=I, seed=7)
    ref = O.layer_fwd_bwd(host["X"], host["topk_idx"], host["topk_w"], host["W_gate"], host["W_up"], host["W_down"],
                          host["dY"])
    for fused in (False, True):
        b = Hh.run_cuda_layer(Hh.device_workload(host), cfg.E, fused_swiglu_bwd=fused)
        for name in ("counts", "offsets", "row_to_pair", "pair_to_row"):
            assert np.array_equal(getattr(b, name).cpu().numpy(), ref[name]), name
        for attr, key in FLOAT_OUTPUTS:
            if not (fused and attr == "dh_act"):
                Hh.assert_close(Hh.to_np64(getattr(b, attr)), ref[key], f"{key} H={H} I={I} fused={fused}")
