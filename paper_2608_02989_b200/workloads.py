"""Seeded synthetic inputs for the verifier-side MoE layer: layer weights, verification
blocks (hidden states + draft-tree depths), commitment tables and residency masks.

This module holds the input recipe only -- none of the method's arithmetic.  The
library, the tests' CPU oracle and the benchmark all draw their inputs from here.
The five configurations take their shapes from the model families the method was
evaluated on (experts, top-k, hidden and intermediate sizes, layer count), blocks
of at most 64 draft-tree nodes, a commitment table that decays with depth, and --
for the Qwen3-30B-A3B-shaped one -- a Zipf(1.1) popularity prior over the experts
entering as a router bias.  Weights are N(0, 0.02), hidden states N(0, 1).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class BlockConfig:
    index: int          # 1-based configuration number; seeds are 1000*index + layer
    name: str
    dtype: str          # "f32" | "bf16": storage type of hidden states and all weights
    hidden: int         # H
    n_experts: int      # E (routed)
    top_k: int          # k
    inter: int          # I (per-expert SwiGLU intermediate)
    n_shared: int       # always-on shared experts (outside selection)
    n_nodes: int        # T
    max_depth: int      # D
    n_layers: int       # L
    p_scale: float      # commitment table p_d = p_scale * p_decay**d
    p_decay: float
    weighting: int      # 0 renormalise over the selected k; 1 raw softmax; 2 softmax over eligible
    zipf_bias: bool = False
    resident_frac: float = 0.0
    level_widths: tuple | None = None   # fixed tree shape (toy config)
    root_certain: bool = False          # toy config: p_0 = 1

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elt_bytes(self):
        return 4 if self.dtype == "f32" else 2

    @property
    def expert_bytes(self):
        return 3 * self.hidden * self.inter * self.elt_bytes

    def seed(self, layer: int) -> int:
        return 0 if self.index == 1 else 1000 * self.index + layer


CONFIGS = {
    1: BlockConfig(1, "toy", "f32", 256, 16, 2, 512, 0, 8, 3, 1, 1.0, 0.8, 0,
                   level_widths=(1, 2, 2, 3), root_certain=True),
    2: BlockConfig(2, "olmoe", "bf16", 2048, 64, 8, 1024, 0, 32, 6, 16, 0.9, 0.75, 1),
    3: BlockConfig(3, "qwen3-30b-a3b", "bf16", 2048, 128, 8, 768, 0, 64, 8, 48, 1.0, 0.85, 0,
                   zipf_bias=True),
    4: BlockConfig(4, "deepseek-v2-lite", "bf16", 2048, 64, 6, 1408, 2, 48, 7, 26, 1.0, 0.8, 1),
    5: BlockConfig(5, "qwen3-235b-a22b", "bf16", 4096, 128, 8, 1536, 0, 64, 8, 94, 1.0, 0.85, 0,
                   resident_frac=0.4),
}


def scaled(cfg: BlockConfig, **kw) -> BlockConfig:
    """A copy with some sizes overridden (reduced cases for CPU tests and profiler captures)."""
    return replace(cfg, **kw)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def commitment_table(cfg: BlockConfig) -> torch.Tensor:
    """p_d for d = 0..D, float32 on the host."""
    p = [cfg.p_scale * cfg.p_decay ** d for d in range(cfg.max_depth + 1)]
    if cfg.root_certain:
        p[0] = 1.0
    return torch.tensor(p, dtype=torch.float32)


def tree_depths(cfg: BlockConfig, layer: int = 0) -> torch.Tensor:
    """Depth of every node, root first, sorted by depth.  Every level 1..D holds at least one
    node; the rest are spread uniformly over the levels (seeded).  int32 on the host."""
    if cfg.level_widths is not None:
        d = [lvl for lvl, w in enumerate(cfg.level_widths) for _ in range(w)]
        return torch.tensor(d, dtype=torch.int32)
    T, D = cfg.n_nodes, cfg.max_depth
    if T == 1:
        return torch.zeros(1, dtype=torch.int32)
    D = min(D, T - 1)
    g = _gen(cfg.seed(0) + 500_000, "cpu")      # one tree per configuration, shared by its layers
    extra = torch.randint(1, D + 1, (T - 1 - D,), generator=g)
    d = torch.cat([torch.zeros(1, dtype=torch.long), torch.arange(1, D + 1), extra])
    return torch.sort(d).values.to(torch.int32)


def batch_tree_depths(cfg: BlockConfig, n_blocks: int):
    """A batch of `n_blocks` verification blocks that together hold cfg.n_nodes nodes (sizes differ by at
    most one node, larger blocks first): returns (offsets [n_blocks+1], depths [T] int32).  Every block is
    a tree of its own, built like tree_depths: root first, every level 1..min(D, size-1) occupied, the
    rest uniform over the levels (seeded per block), sorted by depth."""
    T = cfg.n_nodes
    if not 1 <= n_blocks <= T:
        raise ValueError("n_blocks must be between 1 and the number of nodes")
    sizes = [T // n_blocks + (1 if b < T % n_blocks else 0) for b in range(n_blocks)]
    offsets, depths = [0], []
    for b, n in enumerate(sizes):
        D = min(cfg.max_depth, n - 1)
        g = _gen(cfg.seed(0) + 600_000 + b, "cpu")
        extra = torch.randint(1, D + 1, (n - 1 - D,), generator=g) if n - 1 - D > 0 else torch.zeros(0, dtype=torch.long)
        d = torch.cat([torch.zeros(1, dtype=torch.long), torch.arange(1, D + 1), extra])
        depths.append(torch.sort(d).values.to(torch.int32))
        offsets.append(offsets[-1] + n)
    return offsets, torch.cat(depths)


def hidden_states(cfg: BlockConfig, layer: int, device="cpu") -> torch.Tensor:
    """x [T, H], N(0, 1), independent per layer."""
    g = _gen(cfg.seed(layer) + 100_000, device)
    x = torch.empty(cfg.n_nodes, cfg.hidden, dtype=torch.float32, device=device)
    x.normal_(0.0, 1.0, generator=g)
    return x.to(cfg.torch_dtype)


def layer_weights(cfg: BlockConfig, layer: int, device="cpu", experts: bool = True) -> dict:
    """Router and expert weights of one layer, N(0, 0.02).

    w_router [E,H]; router_bias [E] f32 or None; gate_up [E,2I,H] (rows 0..I-1 gate, I..2I-1 up);
    down [E,H,I]; shared_gate_up [n_shared,2I,H] / shared_down [n_shared,H,I] or None.
    """
    g = _gen(cfg.seed(layer), device)
    dt = cfg.torch_dtype
    E, H, I = cfg.n_experts, cfg.hidden, cfg.inter

    def normal(*shape):
        t = torch.empty(*shape, dtype=dt, device=device)
        t.normal_(0.0, 0.02, generator=g)
        return t

    out = {"w_router": normal(E, H), "router_bias": None, "gate_up": None, "down": None,
           "shared_gate_up": None, "shared_down": None}
    if cfg.zipf_bias:
        perm = torch.randperm(E, generator=_gen(cfg.seed(layer) + 200_000, "cpu"))
        rank = torch.empty(E, dtype=torch.float64)
        rank[perm] = torch.arange(1, E + 1, dtype=torch.float64)
        out["router_bias"] = (-1.1 * torch.log(rank)).to(torch.float32).to(device)
    if experts:
        out["gate_up"] = normal(E, 2 * I, H)
        out["down"] = normal(E, H, I)
        if cfg.n_shared:
            out["shared_gate_up"] = normal(cfg.n_shared, 2 * I, H)
            out["shared_down"] = normal(cfg.n_shared, H, I)
    return out


def resident_mask(cfg: BlockConfig, layer: int) -> torch.Tensor:
    """Bitmask (int32 words, expert e = bit e%32 of word e//32) of the GPU-resident experts:
    the first round(resident_frac*E) entries of a seeded permutation.  All ones when the
    configuration has no offloading."""
    E = cfg.n_experts
    words = (E + 31) // 32
    bits = [0] * words
    if cfg.resident_frac <= 0.0:
        chosen = range(E)
    else:
        perm = torch.randperm(E, generator=_gen(cfg.seed(layer) + 300_000, "cpu"))
        chosen = perm[: int(round(cfg.resident_frac * E))].tolist()
    for e in chosen:
        bits[e // 32] |= 1 << (e % 32)
    return torch.tensor([b - (1 << 32) if b >= (1 << 31) else b for b in bits], dtype=torch.int32)


def weight_bytes_per_layer(cfg: BlockConfig) -> int:
    return (cfg.n_experts + cfg.n_shared) * cfg.expert_bytes + cfg.n_experts * cfg.hidden * cfg.elt_bytes


def describe(cfg: BlockConfig) -> str:
    return (f"C{cfg.index} {cfg.name}: H={cfg.hidden} E={cfg.n_experts} k={cfg.top_k} I={cfg.inter} "
            f"shared={cfg.n_shared} T={cfg.n_nodes} D={cfg.max_depth} L={cfg.n_layers} {cfg.dtype} "
            f"p_d={cfg.p_scale}*{cfg.p_decay}^d expert={cfg.expert_bytes / 1e6:.3f} MB "
            f"layer={weight_bytes_per_layer(cfg) / 1e9:.3f} GB"
            + (f" resident={math.floor(cfg.resident_frac * 100)}%" if cfg.resident_frac else ""))


# ---- MXFP4 expert weights (the GPT-OSS-style storage the paper's offload table mentions) -------------
# Microscaling FP4: blocks of 32 consecutive K elements share a power-of-two scale (one E8M0 byte: 2^(s-127));
# an element is a 4-bit E2M1 code (sign, 2 exponent bits, 1 mantissa bit: 0, 0.5, 1, 1.5, 2, 3, 4, 6).
# This is input preparation (how the synthetic weights are put into that storage), not the method.
E2M1_VALUES = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)


def quantize_mxfp4(w: torch.Tensor):
    """w [..., K] (K a multiple of 32) -> (codes uint8 [..., K] with the 4-bit code of every element,
    scales uint8 [..., K/32]).  Per block: shared exponent = floor(log2(max|w|)) - 2 (2 = the largest E2M1
    exponent), clamped to the E8M0 range; elements are rounded to the nearest E2M1 value (ties to the even
    code) and saturate at +-6.  A block of zeros gets scale 2^-127."""
    if w.shape[-1] % 32 != 0:
        raise ValueError("the last dimension must be a multiple of 32")
    wf = w.detach().to(torch.float32).reshape(*w.shape[:-1], w.shape[-1] // 32, 32)
    amax = wf.abs().amax(dim=-1, keepdim=True)
    exp = torch.floor(torch.log2(torch.clamp(amax, min=2.0 ** -126))) - 2.0
    exp = torch.clamp(exp, -127.0, 127.0)
    exp = torch.where(amax > 0, exp, torch.full_like(exp, -127.0))
    scaled = wf / torch.exp2(exp)
    mag = scaled.abs().clamp(max=6.0)
    # nearest grid point = the number of midpoints passed; at a midpoint take the even code (the midpoint
    # between codes i and i+1 goes up only when i+1 is even)
    best = torch.zeros_like(mag, dtype=torch.uint8)
    for i in range(7):
        mid = 0.5 * (E2M1_VALUES[i] + E2M1_VALUES[i + 1])
        best += ((mag >= mid) if i % 2 == 1 else (mag > mid)).to(torch.uint8)
    codes = (best + 8 * (scaled < 0).to(torch.uint8)).reshape(w.shape)
    scales = (exp.squeeze(-1) + 127.0).to(torch.uint8)
    return codes, scales


def layer_weights_mxfp4(cfg: BlockConfig, layer: int, device="cpu") -> dict:
    """The layer's weights with the routed experts in MXFP4: the bf16 draw of layer_weights, quantised.
    Adds gate_up_codes [E,2I,H] / gate_up_scales [E,2I,H/32] and down_codes [E,H,I] / down_scales [E,H,I/32]
    (uint8); gate_up / down are dropped."""
    w = layer_weights(cfg, layer, device)
    w["gate_up_codes"], w["gate_up_scales"] = quantize_mxfp4(w.pop("gate_up"))
    w["down_codes"], w["down_scales"] = quantize_mxfp4(w.pop("down"))
    w["gate_up"] = w["down"] = None
    return w
