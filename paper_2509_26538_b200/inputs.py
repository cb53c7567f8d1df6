"""Seeded synthetic inputs and the named workload shapes.

This module holds no arithmetic of the method: only shapes, seeds and random
draws, so that the CUDA path and the CPU oracle can be fed the same bytes.
The Flux-shaped workloads stand in for Flux.1-dev activations (24 heads x 128,
512 text tokens, one token per 16x16 pixel patch).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

SEED_BASE = 20250926


@dataclass(frozen=True)
class Workload:
    name: str
    H: int
    W: int
    n_text: int
    batch: int
    heads: int
    head_dim: int
    dtype: str  # "bf16", "fp32" or "fp8" (e4m3 q, k, v; bf16 out)
    tile: int
    shared_region: int
    layer_offset: int
    seed: int

    @property
    def HW(self) -> int:
        return self.H * self.W

    @property
    def S(self) -> int:
        return self.n_text + self.HW

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    # tiny grid, fp32, four layers with offsets 0/16/32/48
    "tiny16": Workload("tiny16", 16, 16, 0, 1, 2, 64, "fp32", 64, 2, 0, SEED_BASE + 1),
    # Flux 1024^2: 64x64 + 512 text
    "flux1024": Workload("flux1024", 64, 64, 512, 1, 24, 128, "bf16", 1024, 8, 512, SEED_BASE + 2),
    # Flux 2048^2: 128x128 + 512 text
    "flux2048": Workload("flux2048", 128, 128, 512, 1, 24, 128, "bf16", 1024, 16, 512, SEED_BASE + 3),
    # stress 4096^2: 256x256 + 512 text
    "flux4096": Workload("flux4096", 256, 256, 512, 1, 24, 128, "bf16", 2048, 32, 1024, SEED_BASE + 5),
}

TINY_LAYER_OFFSETS = (0, 16, 32, 48)
SCHEDULE_LAYERS = 57  # 19 joint + 38 single-stream blocks


def schedule_offset(layer: int, tile: int, HW: int) -> int:
    """Offset of layer `layer` in the full per-step schedule workload."""
    return (layer * tile // 4) % HW


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "fp32": torch.float32, "fp8": torch.float8_e4m3fn}[name]


def make_qkv(wl: Workload, heads: int | None = None, q_gain: float = 1.0):
    """Q, K, V ~ N(0,1) in the ORIGINAL token order, [B, heads, S, D], on the CPU.

    Drawn in float32 from the workload's seed, then rounded to the workload
    dtype.  `heads` draws only the first few heads (same values as the full
    draw is NOT guaranteed; callers use one setting per comparison).
    `q_gain` scales Q before rounding (peaky softmax rows).
    """
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed)
    hh = wl.heads if heads is None else heads
    shape = (wl.batch, hh, wl.S, wl.head_dim)
    dt = torch_dtype(wl.dtype)
    q = (torch.randn(shape, generator=g, dtype=torch.float32) * q_gain).to(dt)
    k = torch.randn(shape, generator=g, dtype=torch.float32).to(dt)
    v = torch.randn(shape, generator=g, dtype=torch.float32).to(dt)
    return q, k, v


def make_smooth_qkv(wl: Workload, heads: int | None = None):
    """Image-like inputs: a low-frequency field of (row, col) plus noise."""
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed + 1000)
    hh = wl.heads if heads is None else heads
    D = wl.head_dim
    dt = torch_dtype(wl.dtype)
    r = torch.arange(wl.H, dtype=torch.float32).view(-1, 1).expand(wl.H, wl.W).reshape(-1) / wl.H
    c = torch.arange(wl.W, dtype=torch.float32).view(1, -1).expand(wl.H, wl.W).reshape(-1) / wl.W
    out = []
    for _ in range(3):
        fr = torch.randn((hh, 1, D), generator=g) * 3.0
        fc = torch.randn((hh, 1, D), generator=g) * 3.0
        ph = torch.rand((hh, 1, D), generator=g) * 6.2831853
        img = torch.sin(fr * r.view(1, -1, 1) + fc * c.view(1, -1, 1) + ph)
        txt = torch.randn((hh, wl.n_text, D), generator=g)
        x = torch.cat([txt, img], dim=1) + 0.25 * torch.randn((hh, wl.S, D), generator=g)
        out.append(x.unsqueeze(0).expand(wl.batch, -1, -1, -1).contiguous().to(dt))
    return tuple(out)


def sample_rows(wl: Workload, n: int, seed: int = 0):
    """A seeded sample of original-order query rows: always includes the first
    and last text token, the first and last image token, and random others."""
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed * 7 + seed)
    fixed = [wl.n_text, wl.S - 1]
    if wl.n_text:
        fixed += [0, wl.n_text - 1]
    extra = torch.randint(0, wl.S, (max(0, n - len(fixed)),), generator=g).tolist()
    rows = sorted(set(fixed + extra))
    return rows
