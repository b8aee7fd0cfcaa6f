"""Seeded synthetic workloads shaped like the paper's models.

This module only makes inputs: shapes, seeds, random tensors and the per-layer
cache-demanding mask.  It contains none of the method's arithmetic (no selection rule,
no attention, no resize), so both the CUDA path and the test oracle may consume what it
produces.  Pretrained weights and ImageNet / GenEval inputs are not available; tensors with
the same shapes and a fixed value distribution stand in for them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Sequence, Tuple

import torch

# Scale side lengths: the 256x256 class-conditional schedule grows from 1x1 to 16x16
# (Sec. 3.2); the 1024x1024 text-to-image schedule ends at 64x64.
SIDES_256 = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)
SIDES_1024 = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)
# 512x512 class-conditional generation (Sec. 5 evaluates a depth-36 model on it): the paper does not
# print that schedule; this is a ten-scale schedule ending at 32x32 (2 240 tokens) of the same kind.
SIDES_512 = (1, 2, 3, 4, 6, 9, 13, 18, 24, 32)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    heads: int
    head_dim: int
    batch: int            # images; rows = 2 * batch (classifier-free guidance doubling)
    sides: Tuple[int, ...]
    n_condensed: int
    n_local: int
    demanding_fraction: float
    seed: int

    @property
    def rows(self) -> int:
        return 2 * self.batch

    @property
    def tokens(self) -> Tuple[int, ...]:
        return tuple(s * s for s in self.sides)

    def n_demanding(self) -> int:
        return int(math.floor(self.demanding_fraction * self.layers + 0.5))

    def demanding_mask(self) -> List[bool]:
        """Seeded permutation of the layers; the first n_demanding of it are cache-demanding."""
        g = torch.Generator(device="cpu")
        g.manual_seed(self.seed * 7919 + 17)
        perm = torch.randperm(self.layers, generator=g).tolist()
        chosen = set(perm[: self.n_demanding()])
        return [i in chosen for i in range(self.layers)]

    def policies(self, full_retention: bool = False) -> List[Tuple[int, int, bool]]:
        mask = self.demanding_mask()
        return [(self.n_condensed, self.n_local, True if full_retention else mask[i])
                for i in range(self.layers)]

    def token_budgets(self) -> List[Tuple[int, int]]:
        """Per-layer (C_bgt, C_cds) in tokens, the way Sec. 5 sets them: C_cds = the condensed scales,
        C_min = C_cds + the penultimate scale (cache-efficient layers), C_max = C_cds + the last two
        scales (cache-demanding layers)."""
        tok = self.tokens
        cds = sum(tok[: self.n_condensed])
        c_min = cds + (tok[-2] if len(tok) > 1 else tok[-1])
        c_max = cds + sum(tok[-2:])
        return [(c_max if dem else c_min, cds) for dem in self.demanding_mask()]

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    # single layer, every element compared with the oracle
    "single": Workload("single", 1, 16, 64, 1, SIDES_256, 2, 2, 0.0, 20251116),
    # VAR-d16-shaped: dim 1024, batch 64
    "var_d16": Workload("var_d16", 16, 16, 64, 64, SIDES_256, 2, 2, 0.5, 20251117),
    # VAR-d30-shaped: dim 1920, batch 256 (the batch the paper reaches only with AMS-KV)
    "var_d30": Workload("var_d30", 30, 30, 64, 256, SIDES_256, 2, 2, 0.3, 20251118),
    # depth-36-shaped 512x512 model: dim 2304 = 36 heads x 64, 36 layers, batch 32
    "var_d36_512": Workload("var_d36_512", 36, 36, 64, 32, SIDES_512, 2, 2, 0.3, 20251120),
    # 1024x1024 text-to-image shaped: dim 2048, head_dim 128, batch 8
    "t2i_1024": Workload("t2i_1024", 32, 16, 128, 8, SIDES_1024, 3, 2, 0.4, 20251119),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal_bf16(shape: Sequence[int], seed: int, device="cpu", std: float = 0.125) -> torch.Tensor:
    """i.i.d. N(0, std^2) values rounded to bf16 (the default std is the configs' N(0,1)/8)."""
    dev = torch.device(device)
    x = torch.randn(tuple(shape), generator=_gen(seed, dev), device=dev, dtype=torch.float32)
    return (x * std).to(torch.bfloat16)


def qkv_for_scale(rows: int, heads: int, tokens: int, head_dim: int, seed: int, scale: int,
                  device="cpu", std: float = 0.125):
    """Q, K, V of one scale, each [rows, heads, tokens, head_dim] bf16, keyed by (seed, scale)."""
    base = int(seed) * 1000 + scale * 3
    shape = (rows, heads, tokens, head_dim)
    return (normal_bf16(shape, base + 0, device, std), normal_bf16(shape, base + 1, device, std),
            normal_bf16(shape, base + 2, device, std))


def peaked_qkv_for_scale(rows: int, heads: int, tokens: int, head_dim: int, seed: int, scale: int,
                         device="cpu", gain: float = 6.0):
    """Like qkv_for_scale but with Q and K large enough that softmax rows are sharply peaked
    (logit spread of several units), which exercises the running-max update of a tiled softmax."""
    q, k, v = qkv_for_scale(rows, heads, tokens, head_dim, seed, scale, device, std=1.0)
    return ((q.float() * gain).to(torch.bfloat16), k, v)


def smooth_field_keys(rows: int, heads: int, sides: Sequence[int], head_dim: int, seed: int,
                      rho: float, device="cpu", std: float = 0.125, n_waves: int = 3) -> List[torch.Tensor]:
    """Per-scale key maps that share a smooth spatial field with weight rho.

    K_s(y, x) = std * (rho * g(u, v) + sqrt(1 - rho^2) * eps_s(y, x)), where (u, v) is the
    pixel centre in [0,1]^2, g is a unit-variance sum of a few low-frequency cosines with
    seeded random phases per (row, head, channel), and eps_s is fresh N(0,1) noise per scale.
    rho = 0 gives independent scales; rho = 0.9 gives strongly correlated adjacent scales.
    Returns a list of [rows, heads, s*s, head_dim] bf16 tensors (raster token order).
    """
    dev = torch.device(device)
    g = _gen(seed * 31 + 5, dev)
    n = rows * heads
    phase = torch.rand((n, 1, head_dim, n_waves), generator=g, device=dev) * (2 * math.pi)
    fy = torch.randint(0, 2, (n, 1, head_dim, n_waves), generator=g, device=dev).float()
    fx = torch.randint(0, 2, (n, 1, head_dim, n_waves), generator=g, device=dev).float()
    out = []
    for si, s in enumerate(sides):
        c = (torch.arange(s, device=dev, dtype=torch.float32) + 0.5) / s
        v, u = torch.meshgrid(c, c, indexing="ij")
        u = u.reshape(1, s * s, 1, 1)
        v = v.reshape(1, s * s, 1, 1)
        waves = torch.cos(math.pi * (fx * u + fy * v) + phase)       # [n, T, D, n_waves]
        field = waves.sum(-1) * math.sqrt(2.0 / n_waves)
        eps = torch.randn((n, s * s, head_dim), generator=g, device=dev)
        k = std * (rho * field + math.sqrt(max(0.0, 1.0 - rho * rho)) * eps)
        out.append(k.to(torch.bfloat16).reshape(rows, heads, s * s, head_dim))
    return out


def growing_logit_qkv(rows: int, heads: int, tokens: int, head_dim: int, seed: int, scale: int,
                      first_level: int = 0, step: int = 8, group: int = 64, device="cpu"):
    """Q, K, V whose attention logits climb by `step` (natural-log units) every `group` key tokens.

    u is a fixed +-1/8 sign vector per (row, head); Q = 8 u + noise/32 and key j = level_j * u + noise/8 with
    level_j = step * (first_level + j // group), so that with a softmax scale of 8 / (head_dim) ... i.e.
    1/8 for 64 channels and 1/16 for 128 ... the logit of key j is level_j plus a small random part.  A tiled
    softmax that walks the keys in order meets a much larger maximum in every tile.  All values are exactly
    representable in bf16 before the noise is added.
    """
    dev = torch.device(device)
    g = _gen(int(seed) * 1000 + scale * 3 + 500, dev)
    sign = (torch.randint(0, 2, (rows, heads, 1, head_dim), generator=g, device=dev).float() * 2 - 1) / 8
    level = step * (first_level + torch.arange(tokens, device=dev) // group).float().reshape(1, 1, tokens, 1)
    noise = lambda: torch.randn((rows, heads, tokens, head_dim), generator=g, device=dev) / 8   # noqa: E731
    q = (8 * sign + noise() / 4).to(torch.bfloat16)
    k = (level * sign + noise()).to(torch.bfloat16)
    v = noise().to(torch.bfloat16)
    return q, k, v
