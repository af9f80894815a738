"""Seeded synthetic inputs for the MoE expert-FFN layer.

This module only draws inputs: activations, weights, upstream gradients and the routing decision
(expert ids and routing weights per token).  It holds none of the layer's arithmetic and is the one
module shared by the CUDA tests/benchmark and the CPU oracle's tests: both sides get the same
bytes.  The router itself (softmax / top-k) is not part of the hot path; it appears here only as
the recipe that produces `topk_idx` / `topk_w`.

The five named configurations stand in for the paper's MoE training workload (a production MoE
stack with routing statistics measured on long-context prompts through a trained router, neither
of which is available offline): they keep the shapes and the load character, from near-uniform
loads to a heavy tail with empty experts.

Value recipe (numpy PCG64, independent stream per (config, tensor)):
  X, dY        ~ N(0,1), rounded to bf16 (round-to-nearest-even)
  W_gate, W_up ~ N(0, std 0.02) [E,H,I];  W_down ~ N(0, std 0.02) [E,I,H]; rounded to bf16
  routing      logits z ~ N(0,1) [T,E] (+ a per-expert bias N(0, std 0.5) for "skew"); the K
               largest logits per token, ties to the lower expert id, slots in descending logit
               order; weights = softmax(z) restricted to the chosen experts and renormalised.
  "zipf"       expert chosen without replacement per token with probability proportional to
               rank^-1.2 over a random expert permutation (Gumbel top-K on log q); the
               `n_empty` least likely ranks get probability zero so that some experts receive
               no tokens at all; weights ~ Dirichlet(1).
  routing weights are computed in fp64, rounded to bf16-representable values and stored as fp32.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class MoeConfig:
    name: str
    T: int
    H: int
    I: int
    E: int
    K: int
    routing: str = "softmax"      # "softmax" | "skew" | "zipf" | "dirichlet_multinomial"
    n_empty: int = 0              # zipf only: ranks that get probability zero
    cfg_id: int = 0

    @property
    def R(self) -> int:
        return self.T * self.K

    @property
    def flops_fwd_bwd(self) -> float:
        """18*R*H*I: forward 6RHI (gate, up, down), backward 12RHI (three dgrads + three wgrads)."""
        return 18.0 * self.R * self.H * self.I


CONFIGS = {
    "tiny": MoeConfig("tiny", T=256, H=256, I=512, E=8, K=2, routing="softmax", cfg_id=1),
    "fine_grained": MoeConfig("fine_grained", T=4096, H=2048, I=1408, E=64, K=6, routing="softmax", cfg_id=2),
    "many_small": MoeConfig("many_small", T=16384, H=2048, I=768, E=128, K=8, routing="skew", cfg_id=3),
    "few_large": MoeConfig("few_large", T=8192, H=4096, I=14336, E=8, K=2, routing="softmax", cfg_id=4),
    "imbalanced": MoeConfig("imbalanced", T=32768, H=4096, I=1536, E=64, K=8, routing="zipf", n_empty=4, cfg_id=5),
}
CONFIG_ORDER = ["tiny", "fine_grained", "many_small", "few_large", "imbalanced"]

# The paper's own weight-gradient workload (section "Production Validation: VeOmni MoE" and its appendix):
# hidden 2880, gate_up width 5760 (I = 2880), 128 experts, top-4, R = 57 768 routed rows whose per-expert counts
# follow Dirichlet(0.24)-multinomial (heavy tail, several empty experts).  14 442 tokens x 4 = 57 768.
CONFIGS["paper_dw1"] = MoeConfig("paper_dw1", T=14442, H=2880, I=2880, E=128, K=4, routing="dirichlet_multinomial",
                                 cfg_id=6)


def round_to_bf16(x) -> np.ndarray:
    """float32 array whose values are the bf16 round-to-nearest-even of x (finite inputs)."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32)


def _rng(seed: int, cfg_id: int, tensor_id: int) -> np.random.Generator:
    return np.random.default_rng([seed, cfg_id, tensor_id])


def _topk_desc(keys: np.ndarray, K: int) -> np.ndarray:
    """Indices of the K largest keys per row, descending, ties to the lower index."""
    order = np.argsort(-keys, axis=1, kind="stable")
    return order[:, :K]


def make_routing(cfg: MoeConfig, seed: int = 0):
    """topk_idx [T,K] int32, topk_w [T,K] float32 (bf16-representable values)."""
    T, E, K = cfg.T, cfg.E, cfg.K
    if cfg.routing in ("softmax", "skew"):
        z = _rng(seed, cfg.cfg_id, 5).standard_normal((T, E))
        if cfg.routing == "skew":
            z = z + 0.5 * _rng(seed, cfg.cfg_id, 6).standard_normal(E)[None, :]
        idx = _topk_desc(z, K)
        zs = np.take_along_axis(z, idx, axis=1)
        p = np.exp(zs - zs.max(axis=1, keepdims=True))
        w = p / p.sum(axis=1, keepdims=True)
    elif cfg.routing == "zipf":
        perm = _rng(seed, cfg.cfg_id, 6).permutation(E)          # perm[rank] = expert id
        live = E - cfg.n_empty
        if live < K:
            raise ValueError("not enough non-empty experts for top-K")
        q = np.zeros(E)
        q[:live] = np.arange(1, live + 1, dtype=np.float64) ** -1.2
        logq = np.full(E, -np.inf)
        logq[perm[:live]] = np.log(q[:live] / q.sum())
        gumbel = _rng(seed, cfg.cfg_id, 5).gumbel(size=(T, E))
        idx = _topk_desc(logq[None, :] + gumbel, K)
        w = _rng(seed, cfg.cfg_id, 7).dirichlet(np.ones(K), size=T)
    elif cfg.routing == "dirichlet_multinomial":
        counts = dirichlet_multinomial_counts(E, T * K, alpha=0.24, seed=seed + cfg.cfg_id)
        return make_routing_from_counts(counts, K, seed)
    else:
        raise ValueError(cfg.routing)
    return idx.astype(np.int32), round_to_bf16(w.astype(np.float32))


def make_router_logits(cfg: MoeConfig, seed: int = 0):
    """Router logits [T,E] float32 for the "softmax" / "skew" workloads: the float32 image of the
    values make_routing draws.  An input for the router entry points only: selection and weights are
    the business of the code under test (and of the oracle), not of this module."""
    if cfg.routing not in ("softmax", "skew"):
        raise ValueError("router logits are defined for the softmax / skew routings only")
    z = _rng(seed, cfg.cfg_id, 5).standard_normal((cfg.T, cfg.E))
    if cfg.routing == "skew":
        z = z + 0.5 * _rng(seed, cfg.cfg_id, 6).standard_normal(cfg.E)[None, :]
    return z.astype(np.float32)


def make_routing_from_counts(counts, K: int, seed: int = 0):
    """A routing with prescribed per-expert row counts (sum must be a multiple of K, and no
    count may exceed the number of tokens): used for adversarial load tests (empty experts at the
    ends, single-row experts, tile-boundary sizes).  Tokens get distinct experts per slot where
    the counts allow it; the construction deals rows round-robin from the largest group.
    Returns topk_idx [T,K] int32 and uniform-ish weights [T,K] float32 (bf16-representable).
    """
    counts = np.asarray(counts, dtype=np.int64)
    R = int(counts.sum())
    if R % K:
        raise ValueError("sum(counts) must be a multiple of K")
    T = R // K
    # column-major fill of a [T,K] table from the expert list sorted by expert: token t gets
    # entries t, t+T, t+2T, ... so a token meets the same expert twice only if a count exceeds T.
    flat = np.repeat(np.arange(counts.size), counts)
    idx = flat.reshape(K, T).T.copy()
    rng = _rng(seed, 99, R)
    rows = rng.permutation(T)
    idx = idx[rows]
    w = rng.dirichlet(np.ones(K), size=T)
    return idx.astype(np.int32), round_to_bf16(w.astype(np.float32))


def make_tensors(cfg: MoeConfig, seed: int = 0):
    """Host (numpy) inputs: float32 arrays holding bf16-representable values."""
    T, H, I, E = cfg.T, cfg.H, cfg.I, cfg.E
    c = cfg.cfg_id
    X = round_to_bf16(_rng(seed, c, 0).standard_normal((T, H), dtype=np.float32))
    Wg = round_to_bf16(0.02 * _rng(seed, c, 1).standard_normal((E, H, I), dtype=np.float32))
    Wu = round_to_bf16(0.02 * _rng(seed, c, 2).standard_normal((E, H, I), dtype=np.float32))
    Wd = round_to_bf16(0.02 * _rng(seed, c, 3).standard_normal((E, I, H), dtype=np.float32))
    dY = round_to_bf16(_rng(seed, c, 4).standard_normal((T, H), dtype=np.float32))
    return dict(X=X, W_gate=Wg, W_up=Wu, W_down=Wd, dY=dY)


def make_workload(cfg: MoeConfig, seed: int = 0):
    """Everything one layer call needs, on the host."""
    d = make_tensors(cfg, seed)
    d["topk_idx"], d["topk_w"] = make_routing(cfg, seed)
    return d


def make_workload_device(cfg: MoeConfig, device, seed: int = 0):
    """The same workload with the large float tensors drawn on the device (torch's seeded device
    generator) to keep set-up time short at the full-size configurations.  Routing is always
    drawn on the host with make_routing.  Values follow the same distributions; the bytes differ
    from make_workload's.  Returns torch tensors (bf16 / int32 / float32) on `device`.
    """
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(1000 * (seed + 1) + cfg.cfg_id)
    T, H, I, E = cfg.T, cfg.H, cfg.I, cfg.E

    def randn(shape, std):
        out = torch.empty(shape, dtype=torch.bfloat16, device=device)
        # draw in slabs to bound the fp32 temporary
        flat = out.view(-1)
        step = 1 << 28
        for s in range(0, flat.numel(), step):
            n = min(step, flat.numel() - s)
            flat[s:s + n] = (torch.randn(n, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
        return out

    idx, w = make_routing(cfg, seed)
    return dict(
        X=randn((T, H), 1.0), W_gate=randn((E, H, I), 0.02), W_up=randn((E, H, I), 0.02),
        W_down=randn((E, I, H), 0.02), dY=randn((T, H), 1.0),
        topk_idx=torch.from_numpy(idx).to(device), topk_w=torch.from_numpy(w).to(device))


def dirichlet_multinomial_counts(E: int, R: int, alpha: float = 0.24, seed: int = 0) -> np.ndarray:
    """Per-expert row counts K_e with p ~ Dirichlet(alpha*1_E), (K_1..K_E) ~ Multinomial(R, p):
    the paper's routing-imbalance model for its weight-gradient benchmark (heavy tail, several
    empty experts for small alpha)."""
    rng = _rng(seed, 77, E)
    p = rng.dirichlet(np.full(E, alpha))
    return rng.multinomial(R, p).astype(np.int64)
