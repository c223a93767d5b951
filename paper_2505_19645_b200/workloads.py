"""Seeded synthetic inputs for the MoE verify layer.

This module holds NONE of the method's arithmetic: it only names the layer shapes the
benchmark sweeps and draws the random tensors (weights, token activations, router
matrix, optional popularity bias) that both the CUDA path and the CPU oracle are fed.

Recipe (stand-in for the paper's Sec. 4 workloads, whose prompt sets and trained weights
are not available; the FFN layer sees only the token count and the routing statistics,
which Sec. 3.2 itself models as uniform):
  expert / shared-expert weights  bf16 ~ N(0, 0.02)
  shared scalar gate vector       bf16 ~ N(0, 0.02)
  router matrix                   fp32 ~ N(0, 0.02)
  token activations               bf16 ~ N(0, 1)
With iid Gaussian router rows the logits of one token are exchangeable across experts, so
its top-k set is uniform over the k-subsets ("balanced routing", the uniform-activation
assumption behind Eq. N(t)).  The Zipf variant adds a router bias b_e = beta * ln p_e
with p_e ~ rank^-s over a seeded random ranking and beta chosen so that the bias competes
with the logit noise (std 0.02*sqrt(H)) on a Gumbel scale; it is "Zipf-like", not exact.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, asdict

import torch

SCORE_SOFTMAX = 0
SCORE_SIGMOID = 1


@dataclass(frozen=True)
class LayerShape:
    name: str
    hidden: int          # H
    n_experts: int       # E
    top_k: int           # k
    inter: int           # I
    shared_inter: int    # I_s, 0 = no shared expert
    score_fn: int        # SCORE_SOFTMAX / SCORE_SIGMOID
    renormalize: int     # 1: top-k weights divided by their sum
    shared_gate: int     # 1: shared expert scaled by sigmoid(x . w_sg)
    routed_scale: float = 1.0

    def as_dict(self) -> dict:
        return asdict(self)


# The five layer shapes of the benchmark sweep, with their (B, gamma) grids.
CONFIGS = {
    "tiny": LayerShape("tiny", 256, 8, 2, 512, 0, SCORE_SOFTMAX, 1, 0),
    "qwen1.5-moe-a2.7b": LayerShape("qwen1.5-moe-a2.7b", 2048, 60, 4, 1408, 5632,
                                    SCORE_SOFTMAX, 0, 1),
    "qwen2-57b-a14b": LayerShape("qwen2-57b-a14b", 3584, 64, 8, 2560, 20480,
                                 SCORE_SOFTMAX, 0, 1),
    "mixtral-8x7b": LayerShape("mixtral-8x7b", 4096, 8, 2, 14336, 0, SCORE_SOFTMAX, 1, 0),
    "deepseek-v3": LayerShape("deepseek-v3", 7168, 256, 8, 2048, 2048, SCORE_SIGMOID, 1, 0),
}
CONFIG_ORDER = ["tiny", "qwen1.5-moe-a2.7b", "qwen2-57b-a14b", "mixtral-8x7b", "deepseek-v3"]

GRIDS = {
    "tiny": ([4], [3]),
    "qwen1.5-moe-a2.7b": ([1, 4, 16, 32, 64, 128], [0, 1, 2, 3, 4]),
    "qwen2-57b-a14b": ([1, 8, 32, 64, 128, 256], [0, 1, 2, 3, 4]),
    "mixtral-8x7b": ([1, 4, 16, 64, 256], [0, 2, 4]),
    "deepseek-v3": ([1, 16, 64, 128, 256, 512], [0, 1, 3, 5]),
}


# Sparsity sweep on one shape (Sec. 4.3 varies the experts per token K of the Qwen2-57B-A14B
# model, at draft lengths 2 and 4, over these 19 batch sizes).  The paper does not list its
# six K values; these six span rho = K/E from 1/64 to 1/4 and include the model's own K = 8.
SPARSITY_BATCHES = [1, 2, 4, 8, 12, 16, 20, 24, 28, 32, 36, 40, 44, 48, 52, 56, 60, 80, 100]
SPARSITY_GAMMAS = [0, 2, 4]      # gamma = 0 is the denominator T(B, 0) of the cost ratio
SPARSITY_TOP_KS = [1, 2, 4, 8, 12, 16]


def with_top_k(shape: LayerShape, top_k: int) -> LayerShape:
    """The same layer with K experts per token (a run-time parameter of the routing)."""
    d = shape.as_dict()
    d.update(name="%s-k%d" % (shape.name, top_k), top_k=top_k)
    return LayerShape(**d)


def dense_contrast(shape: LayerShape) -> LayerShape:
    """The rho = 1 limit of Sec. 3.3 with the same active parameters per token: one routed
    expert of width K*I that every token uses (plus the unchanged shared expert)."""
    d = shape.as_dict()
    d.update(name="%s-dense" % shape.name, n_experts=1, top_k=1, inter=shape.top_k * shape.inter)
    return LayerShape(**d)


def config_seed(name: str) -> int:
    """Weight seed of a config: 0 for the tiny config, 1000*index otherwise."""
    return 1000 * CONFIG_ORDER.index(name)


def point_seed(name: str, B: int, gamma: int) -> int:
    """Activation seed of one (B, gamma) sweep point of a config."""
    Bs, gs = GRIDS[name]
    ib = Bs.index(B) if B in Bs else len(Bs) + B
    ig = gs.index(gamma) if gamma in gs else len(gs) + gamma
    return config_seed(name) + 10 * ib + ig


def _randn(shape, std, dtype, gen, device):
    # drawn in fp32 on the generator's device, then cast: the same tensor reaches both sides
    t = torch.empty(shape, dtype=torch.float32, device=device)
    t.normal_(0.0, std, generator=gen)
    return t.to(dtype)


def make_weights(shape: LayerShape, seed: int, device="cpu", zipf_s: float | None = None) -> dict:
    """Draw every weight tensor of one layer.  Keys absent from the layer are None."""
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    H, E, I, Is = shape.hidden, shape.n_experts, shape.inter, shape.shared_inter
    w = {
        "w_router": _randn((E, H), 0.02, torch.float32, gen, device),
        "router_bias": None,
        "w_gate": None, "w_up": None, "w_down": None,
        "ws_gate": None, "ws_up": None, "ws_down": None, "w_shared_gate": None,
    }
    # expert by expert so that the fp32 staging buffer stays small for the large shapes
    for key, shp in (("w_gate", (I, H)), ("w_up", (I, H)), ("w_down", (H, I))):
        full = torch.empty((E,) + shp, dtype=torch.bfloat16, device=device)
        for e in range(E):
            full[e] = _randn(shp, 0.02, torch.bfloat16, gen, device)
        w[key] = full
    if Is > 0:
        w["ws_gate"] = _randn((Is, H), 0.02, torch.bfloat16, gen, device)
        w["ws_up"] = _randn((Is, H), 0.02, torch.bfloat16, gen, device)
        w["ws_down"] = _randn((H, Is), 0.02, torch.bfloat16, gen, device)
        if shape.shared_gate:
            w["w_shared_gate"] = _randn((H,), 0.02, torch.bfloat16, gen, device)
    if zipf_s is not None:
        w["router_bias"] = zipf_router_bias(E, H, zipf_s, seed, device)
    return w


def zipf_router_bias(E: int, H: int, s: float, seed: int, device="cpu") -> torch.Tensor:
    """Router bias that skews expert popularity towards p_e ~ rank_e^-s (seeded ranking)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed + 7919)
    rank = torch.randperm(E, generator=gen).to(torch.float64) + 1.0
    p = rank.pow(-s)
    p = p / p.sum()
    beta = 0.02 * math.sqrt(H) * math.sqrt(6.0) / math.pi
    return (beta * p.log()).to(torch.float32).to(device)


def make_tokens(shape: LayerShape, T: int, seed: int, device="cpu") -> torch.Tensor:
    """Token activations x[T, H], bf16 ~ N(0, 1)."""
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed + 104729)
    return _randn((T, shape.hidden), 1.0, torch.bfloat16, gen, device)


def small_shape(name: str, hidden: int, n_experts: int, top_k: int, inter: int,
                shared_inter: int = 0, score_fn: int = SCORE_SOFTMAX, renormalize: int = 1,
                shared_gate: int = 0, routed_scale: float = 1.0) -> LayerShape:
    """Ad-hoc shape for tests."""
    return LayerShape(name, hidden, n_experts, top_k, inter, shared_inter, score_fn,
                      renormalize, shared_gate, routed_scale)
