"""Seeded synthetic inputs shaped like the paper's MoE workloads.

This module only draws random numbers and names shapes: it holds none of the
method's arithmetic (no quantizer, no router, no FFN), so both the CUDA path and
the CPU oracle may be fed from it.  The same bytes go to both sides: a tensor is
generated once, on whichever device is asked for, and copied to the other side.

Layer shapes follow Table 1 of the paper (8 experts top-2; 60+4 / 128+1 style
fine-grained layers with always-on shared experts); hidden and FFN sizes are the
public model shapes.  Real checkpoints and evaluation corpora are not used: these
draws stand in for them.
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np
import torch

KINDS = ("gate", "up", "down")
BITS = (16, 8, 4, 3, 2)
GROUP = 128


@dataclass(frozen=True)
class LayerConfig:
    name: str
    n_experts: int
    top_k: int
    hidden: int
    ffn: int
    tokens: int
    n_shared: int = 0
    n_layers: int = 1
    routing: str = "normal"          # "normal" | "zipf" | "gumbel"
    zipf_a: float = 0.0
    bit_rule: str = "iid5"           # see assign_bits
    seed: int = 0

    @property
    def n_blocks_per_layer(self) -> int:
        return (self.n_experts + self.n_shared) * 3

    def block_shape(self, kind: int) -> Tuple[int, int]:
        """(rows = output features, cols = input features) of a gate / up / down block."""
        return (self.hidden, self.ffn) if kind == 2 else (self.ffn, self.hidden)


CONFIGS: Dict[str, LayerConfig] = {
    # configs[0]: tiny layer the oracle finishes in well under a second
    "tiny": LayerConfig("tiny", 8, 2, 256, 512, 16, routing="normal", bit_rule="iid5"),
    "tiny_cover": LayerConfig("tiny_cover", 8, 2, 256, 512, 16, routing="normal", bit_rule="cycle5"),
    # configs[1]: 8-expert top-2 decode, batch 64, Zipf(1.1) popularity, 25/25/30/10/10 % bit mix
    "mixtral_decode": LayerConfig("mixtral_decode", 8, 2, 4096, 14336, 64, routing="zipf", zipf_a=1.1,
                                  bit_rule="mix_25_25_30_10_10"),
    # configs[2]: 64 routed top-6 + 2 shared, batch 256, Zipf(1.2); int4 except 10 % fp16 / 20 % int2
    "finegrained_decode": LayerConfig("finegrained_decode", 64, 6, 2048, 1408, 256, n_shared=2, routing="zipf",
                                      zipf_a=1.2, bit_rule="int4_10fp16_20int2"),
    # configs[3]: 8-expert top-2 prefill, 4096 tokens, uniform-random routing, bits from {16,8,4}
    "mixtral_prefill": LayerConfig("mixtral_prefill", 8, 2, 4096, 14336, 4096, routing="gumbel", bit_rule="iid3"),
    # latency decode (Table 3 of the paper: batch 1 and batch 4) on a 60 routed top-4 + 4 shared layer
    "latency_b1": LayerConfig("latency_b1", 60, 4, 2048, 1408, 1, n_shared=4, routing="normal",
                              bit_rule="mix_25_25_30_10_10"),
    "latency_b4": LayerConfig("latency_b4", 60, 4, 2048, 1408, 4, n_shared=4, routing="normal",
                              bit_rule="mix_25_25_30_10_10"),
    # many small experts (Table 1: 128 routed + 1 shared, top-8); hidden and FFN sizes are stand-ins
    "manyexpert_decode": LayerConfig("manyexpert_decode", 128, 8, 2048, 768, 64, n_shared=1, routing="zipf",
                                     zipf_a=1.2, bit_rule="int4_10fp16_20int2"),
    # configs[4]: 32 stacked layers, all fp16 at start, 1/3 of the blocks demoted 16->4->2 under load
    "demote_under_load": LayerConfig("demote_under_load", 8, 2, 4096, 14336, 64, n_layers=32, routing="zipf",
                                     zipf_a=1.1, bit_rule="all16"),
}


def _seed(*parts) -> int:
    h = hashlib.sha256(("/".join(str(p) for p in parts)).encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 62) - 1)


def _gen(device, *parts) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*parts))
    return g


def block_weights(cfg: LayerConfig, layer: int, expert: int, kind: int, device="cpu") -> torch.Tensor:
    """fp16 [rows, cols]: N(0, 0.02^2), an independent 0.1 % of entries multiplied by 10."""
    rows, cols = cfg.block_shape(kind)
    g = _gen(device, "w", cfg.seed, cfg.name, layer, expert, kind)
    w = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * 0.02
    mask = torch.rand(rows, cols, generator=g, device=device, dtype=torch.float32) < 0.001
    w = torch.where(mask, w * 10.0, w)
    return w.to(torch.float16)


def activations(cfg: LayerConfig, layer: int = 0, step: int = 0, device="cpu", tokens: int = 0) -> torch.Tensor:
    """fp16 [T, H] ~ N(0, 1)."""
    T = tokens or cfg.tokens
    g = _gen(device, "x", cfg.seed, cfg.name, layer, step, T)
    return torch.randn(T, cfg.hidden, generator=g, device=device, dtype=torch.float32).to(torch.float16)


def router_logits(cfg: LayerConfig, layer: int = 0, step: int = 0, device="cpu", tokens: int = 0) -> torch.Tensor:
    """fp32 [T, E].  "normal": N(0,1).  "gumbel": i.i.d. Gumbel(0,1), i.e. uniform-random top-k.
    "zipf": ln p_pi(e) + Gumbel(0,1) with p_r ~ r^-a and pi a seeded permutation of the experts, so that
    top-1 frequencies are Zipf and top-k is sampling without replacement."""
    T = tokens or cfg.tokens
    E = cfg.n_experts
    g = _gen(device, "l", cfg.seed, cfg.name, layer, step, T)
    if cfg.routing == "normal":
        return torch.randn(T, E, generator=g, device=device, dtype=torch.float32)
    u = torch.rand(T, E, generator=g, device=device, dtype=torch.float64).clamp_(1e-300, 1.0 - 1e-16)
    gum = -torch.log(-torch.log(u))
    if cfg.routing == "gumbel":
        return gum.to(torch.float32)
    if cfg.routing == "zipf":
        rng = np.random.default_rng(_seed("pi", cfg.seed, cfg.name, layer))
        pi = rng.permutation(E)                       # rank of expert e is pi[e] + 1
        p = (pi + 1.0) ** (-cfg.zipf_a)
        p = p / p.sum()
        logp = torch.from_numpy(np.log(p)).to(device)
        return (gum + logp[None, :]).to(torch.float32)
    raise ValueError(cfg.routing)


def assign_bits(cfg: LayerConfig, layer: int = 0) -> np.ndarray:
    """Committed bitwidth q_i of every block of one layer: int array [(E + n_shared), 3]."""
    nb_routed = cfg.n_experts * 3
    rng = np.random.default_rng(_seed("bits", cfg.seed, cfg.name, layer))
    if cfg.bit_rule == "iid5":
        routed = rng.choice(BITS, size=nb_routed)
    elif cfg.bit_rule == "cycle5":
        routed = np.array([BITS[n % 5] for n in range(nb_routed)])
    elif cfg.bit_rule == "iid3":
        routed = rng.choice((16, 8, 4), size=nb_routed)
    elif cfg.bit_rule == "all16":
        routed = np.full(nb_routed, 16)
    elif cfg.bit_rule.startswith("uniform"):
        routed = np.full(nb_routed, int(cfg.bit_rule[len("uniform"):]))
    elif cfg.bit_rule == "mix_25_25_30_10_10":
        shares = np.array([0.25, 0.25, 0.30, 0.10, 0.10]) * nb_routed
        counts = np.floor(shares).astype(int)
        rem = shares - counts
        for i in np.argsort(-rem, kind="stable")[: nb_routed - counts.sum()]:
            counts[i] += 1
        pool = np.repeat(np.array(BITS), counts)
        routed = pool[rng.permutation(nb_routed)]
    elif cfg.bit_rule == "int4_10fp16_20int2":
        n16 = int(0.10 * nb_routed)
        n2 = int(0.20 * nb_routed)
        pool = np.array([16] * n16 + [2] * n2 + [4] * (nb_routed - n16 - n2))
        order = rng.permutation(nb_routed)
        routed = np.empty(nb_routed, int)
        routed[order] = pool
    else:
        raise ValueError(cfg.bit_rule)
    shared = np.full(cfg.n_shared * 3, 16)           # shared experts stay fp16 and are never demoted
    return np.concatenate([routed, shared]).astype(np.int32).reshape(cfg.n_experts + cfg.n_shared, 3)


def demote_schedule(cfg: LayerConfig, fraction: float = 1.0 / 3.0) -> List[Tuple[int, int, int]]:
    """Seeded list of (layer, expert, kind) blocks to demote (routed experts only), 1/3 of all blocks."""
    n = cfg.n_layers * cfg.n_experts * 3
    rng = np.random.default_rng(_seed("demote", cfg.seed, cfg.name))
    pick = rng.permutation(n)[: int(round(n * fraction))]
    out = []
    for b in pick:
        layer, rest = divmod(int(b), cfg.n_experts * 3)
        expert, kind = divmod(rest, 3)
        out.append((layer, expert, kind))
    return out


def zipf_reference_probs(cfg: LayerConfig, layer: int = 0) -> np.ndarray:
    """Top-1 selection probability of every expert under the "zipf" rule (for tests of the generator)."""
    rng = np.random.default_rng(_seed("pi", cfg.seed, cfg.name, layer))
    pi = rng.permutation(cfg.n_experts)
    p = (pi + 1.0) ** (-cfg.zipf_a)
    return p / p.sum()
