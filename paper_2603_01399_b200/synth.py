"""Seeded synthetic inputs for the quantised verification pass.

This module only *draws numbers and lays out shapes*.  It holds none of the
method's arithmetic (no quantisation, no forward pass, no acceptance rule):
the CPU oracle and the CUDA path are each handed the very same bytes produced
here and neither of them imports the other.

Workload shapes follow the paper's experimental setup (Section 4.1: a
Qwen3-8B-class decoder, draft lengths gamma in 3..9) with random-init weights;
the paper's datasets and trained checkpoints are not used.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import torch


@dataclasses.dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    qk_norm: bool
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def qkv_dim(self) -> int:
        return self.q_dim + 2 * self.kv_dim

    def linear_shapes(self):
        """(name, N, K) of the four per-layer matrices and the LM head."""
        return [
            ("qkv", self.qkv_dim, self.hidden),
            ("o", self.hidden, self.q_dim),
            ("gateup", 2 * self.ffn, self.hidden),
            ("down", self.hidden, self.ffn),
            ("lm_head", self.vocab, self.hidden),
        ]

    def weight_elems(self) -> int:
        per_layer = sum(n * k for nm, n, k in self.linear_shapes() if nm != "lm_head")
        return self.n_layers * per_layer + self.vocab * self.hidden


SHAPES = {
    "tiny": ModelShape("tiny", 2, 256, 4, 2, 64, 688, 1024, False),
    "tiny_qknorm": ModelShape("tiny_qknorm", 2, 256, 4, 2, 64, 688, 1024, True),
    "qwen3_8b": ModelShape("qwen3_8b", 36, 4096, 32, 8, 128, 12288, 151936, True),
    "qwen3_14b": ModelShape("qwen3_14b", 40, 5120, 40, 8, 128, 17408, 151936, True),
}

_KIND_IDS = {
    "embed": 1, "attn_norm": 2, "qkv": 3, "q_norm": 4, "k_norm": 5, "o": 6,
    "mlp_norm": 7, "gateup": 8, "down": 9, "final_norm": 10, "lm_head": 11,
    "kv_k": 12, "kv_v": 13, "tokens": 14, "draft": 15, "x": 16, "act_absmax": 17,
}


def sub_seed(seed: int, kind: str, layer: int = 0) -> int:
    """A distinct generator seed per (seed, tensor kind, layer)."""
    return (seed * 1_000_003 + _KIND_IDS[kind] * 10_007 + layer * 101 + 17) % (2**63 - 1)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def normal_bf16(shape, std: float, seed: int, device="cpu") -> torch.Tensor:
    """N(0, std) drawn in fp32 and rounded to bf16."""
    g = _gen(seed, device)
    t = torch.empty(shape, dtype=torch.float32, device=device)
    t.normal_(0.0, std, generator=g)
    return t.to(torch.bfloat16)


def uniform_bf16(shape, lo: float, hi: float, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    t = torch.empty(shape, dtype=torch.float32, device=device)
    t.uniform_(lo, hi, generator=g)
    return t.to(torch.bfloat16)


def uniform_tokens(shape, vocab: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return torch.randint(0, vocab, shape, generator=g, device=device, dtype=torch.int64).to(torch.int32)


def matrix(shape: ModelShape, kind: str, layer: int, seed: int = 0, device="cpu") -> torch.Tensor:
    """bf16 master weight [N][K] ~ N(0, 0.02) for one linear layer."""
    dims = {nm: (n, k) for nm, n, k in shape.linear_shapes()}
    n, k = dims[kind]
    return normal_bf16((n, k), 0.02, sub_seed(seed, kind, layer), device)


def embedding(shape: ModelShape, seed: int = 0, device="cpu") -> torch.Tensor:
    return normal_bf16((shape.vocab, shape.hidden), 0.02, sub_seed(seed, "embed"), device)


def gain(shape: ModelShape, kind: str, layer: int, seed: int = 0, device="cpu") -> torch.Tensor:
    """Norm gain ~ U(0.5, 1.5) so that a dropped gain shows up in parity."""
    n = shape.head_dim if kind in ("q_norm", "k_norm") else shape.hidden
    return uniform_bf16((n,), 0.5, 1.5, sub_seed(seed, kind, layer), device)


def activation_absmax(shape: ModelShape, kind: str, layer: int, seed: int = 0, device="cpu") -> torch.Tensor:
    """Stand-in for the calibration statistic max|X_j| of a linear layer's input (fp32 [K]): most channels
    ~ U(0.5, 4), about one in a hundred an outlier 20 times larger - the "systematic outliers in specific
    activation channels" that smoothing is there for (Section 3.2)."""
    dims = {nm: k for nm, _, k in shape.linear_shapes()}
    k = dims[kind]
    g = _gen(sub_seed(seed, "act_absmax", layer) + 7919 * _KIND_IDS[kind], device)
    base = torch.empty(k, dtype=torch.float32, device=device).uniform_(0.5, 4.0, generator=g)
    outlier = torch.rand(k, generator=g, device=device) < 0.01
    return torch.where(outlier, base * 20.0, base)


def kv_prefix(shape: ModelShape, batch: int, s_max: int, seed: int = 1, device="cpu"):
    """bf16 K and V caches [L][B][Hkv][S_max][D] ~ N(0,1) (all slots filled)."""
    dims = (shape.n_layers, batch, shape.n_kv_heads, s_max, shape.head_dim)
    k = normal_bf16(dims, 1.0, sub_seed(seed, "kv_k"), device)
    v = normal_bf16(dims, 1.0, sub_seed(seed, "kv_v"), device)
    return k, v


def corrupt_draft(greedy: torch.Tensor, p: float, vocab: int, seed: int) -> torch.Tensor:
    """Replace each draft position by a uniform-random token with probability p."""
    g = _gen(sub_seed(seed, "draft"), "cpu")
    greedy = greedy.cpu().to(torch.int32)
    flip = torch.rand(greedy.shape, generator=g) < p
    rnd = torch.randint(0, vocab, greedy.shape, generator=g, dtype=torch.int64).to(torch.int32)
    return torch.where(flip, rnd, greedy)


def chain_parents(t: int) -> List[int]:
    return [-1] + list(range(t - 1))


def tree_parents_16() -> List[int]:
    """Root + 16 candidate nodes, depth 4: four children of the root; the first
    two of those have two children each; every deeper node has one child."""
    parents = [-1]
    d1 = []
    for _ in range(4):
        d1.append(len(parents)); parents.append(0)
    d2 = []
    for p in d1[:2]:
        for _ in range(2):
            d2.append(len(parents)); parents.append(p)
    d3 = []
    for p in d2:
        d3.append(len(parents)); parents.append(p)
    for p in d3:
        parents.append(p)
    assert len(parents) == 17
    return parents


def tree_parents_full(branching=(4, 2, 1, 1)) -> List[int]:
    """Full product tree for the given per-depth branching (28 nodes for 4,2,1,1)."""
    parents = [-1]
    frontier = [0]
    for br in branching:
        nxt = []
        for p in frontier:
            for _ in range(br):
                nxt.append(len(parents)); parents.append(p)
        frontier = nxt
    return parents


def depths(parents: List[int]) -> List[int]:
    d = []
    for i, p in enumerate(parents):
        d.append(0 if p < 0 else d[p] + 1)
    return d


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
