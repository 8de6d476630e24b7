"""Seeded synthetic workloads for the shifted-window attention block.

This module is the one piece shared by the CPU oracle's tests and the CUDA path's
tests: it names the five benchmark configurations and draws their inputs from
seeded generators.  It holds none of the method's arithmetic (no routing, no
attention, no bias indexing) so that the two implementations stay independent.

Inputs stand in for projected, normalised Swin-block activations on the
Wenhai-shaped token grids (the paper's 2041 x 4320 field at patch 4 and patch 2,
Section VII-A): Q, K, V and the upstream gradient dO are i.i.d. N(0, 1) rounded to
bf16 in the contiguous [B, H, W, heads, head_dim] layout; the relative-position
bias table is i.i.d. N(0, std 0.02) fp32 of shape [(2w-1)^2, heads].
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import torch

SEED_BASE = 20260815


@dataclass(frozen=True)
class SwinConfig:
    """One shifted-window attention problem (grid, window, heads)."""

    name: str
    B: int
    H: int           # token rows (latitude)
    W: int           # token columns (longitude)
    heads: int
    head_dim: int
    window: int
    shift_h: int
    shift_w: int
    periodic_h: int = 0   # latitude is not periodic
    periodic_w: int = 1   # longitude is periodic
    backward: bool = True
    index: int = 0

    @property
    def tokens(self) -> int:
        return self.B * self.H * self.W

    @property
    def bias_rows(self) -> int:
        return (2 * self.window - 1) ** 2

    def as_dict(self) -> dict:
        return asdict(self)


CONFIGS = {
    "cfg1": SwinConfig("cfg1", 1, 32, 64, 3, 32, 8, 4, 4, backward=False, index=1),
    "cfg2": SwinConfig("cfg2", 1, 128, 256, 6, 32, 8, 4, 4, index=2),
    "cfg3": SwinConfig("cfg3", 1, 510, 1080, 12, 32, 16, 8, 8, index=3),   # Wenhai-shaped, patch 4
    "cfg4": SwinConfig("cfg4", 1, 256, 512, 12, 64, 32, 16, 16, index=4),  # large window
    "cfg5": SwinConfig("cfg5", 2, 1020, 2160, 8, 32, 14, 7, 7, index=5),   # fine patch, batch 2
    # The paper's own model shapes (Table V: 128 channels per head; patch 4, sampling factor 2 on the field padded to
    # 2304 x 4352, i.e. a 288 x 544 token grid in the Transformer blocks, Section VII-B): small, medium and large model.
    "tv_small": SwinConfig("tv_small", 1, 288, 544, 8, 128, 8, 4, 4, index=6),
    "tv_medium": SwinConfig("tv_medium", 1, 288, 544, 32, 128, 8, 4, 4, index=7),
    "tv_large": SwinConfig("tv_large", 1, 288, 544, 64, 128, 32, 16, 16, index=8),
    # The window-assignment study's largest window (Section VII-E: small model, w = 128; the 2041 x 4320 field at
    # patch 4 and sampling factor 2 padded to a 2 x 5 grid of 128 x 128 windows, i.e. 256 x 640 tokens)
    "tv_small_w128": SwinConfig("tv_small_w128", 1, 256, 640, 8, 128, 128, 64, 64, index=9),
    # A 3 x 5-window slice of the large model's block (same heads, head dim, window, shift): 2.3 GB on the device
    # with gradients, the size a full-counter profiler capture of the head-dim-128 tcgen05 kernels is taken on
    "tv_large_slice": SwinConfig("tv_large_slice", 1, 96, 160, 64, 128, 32, 16, 16, index=10),
    # One row of three 128 x 128 windows of the window-assignment study's block (same heads, head dim, window, shift):
    # 0.9 GB on the device with gradients, for profiler captures of the tcgen05 kernels at window side 128
    "tv_small_w128_slice": SwinConfig("tv_small_w128_slice", 1, 128, 384, 8, 128, 128, 64, 64, index=11),
}

TENSOR_INDEX = {"q": 0, "k": 1, "v": 2, "do": 3, "bias": 4}


def seed_for(cfg: SwinConfig, tensor: str, extra: int = 0) -> int:
    return SEED_BASE + 1000 * cfg.index + TENSOR_INDEX[tensor] + 100 * extra


def make_activation(cfg: SwinConfig, tensor: str, device: str = "cpu", extra: int = 0) -> torch.Tensor:
    """bf16 [B, H, W, heads, head_dim] ~ N(0, 1), drawn on `device` from its seeded generator."""
    g = torch.Generator(device=device)
    g.manual_seed(seed_for(cfg, tensor, extra))
    shape = (cfg.B, cfg.H, cfg.W, cfg.heads, cfg.head_dim)
    n = cfg.tokens * cfg.heads * cfg.head_dim
    if n <= (1 << 28):
        return torch.randn(shape, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    # large tensors: draw per batch sample so the fp32 staging buffer stays bounded
    out = torch.empty(shape, device=device, dtype=torch.bfloat16)
    for b in range(cfg.B):
        out[b].copy_(torch.randn(shape[1:], generator=g, device=device, dtype=torch.float32))
    return out


def make_bias_table(cfg: SwinConfig, device: str = "cpu", extra: int = 0) -> torch.Tensor:
    """fp32 [(2w-1)^2, heads] ~ N(0, std 0.02)."""
    g = torch.Generator(device=device)
    g.manual_seed(seed_for(cfg, "bias", extra))
    return 0.02 * torch.randn((cfg.bias_rows, cfg.heads), generator=g, device=device, dtype=torch.float32)


def make_inputs(cfg: SwinConfig, device: str = "cpu", extra: int = 0) -> dict:
    """All inputs of one forward(+backward) step."""
    out = {t: make_activation(cfg, t, device, extra) for t in ("q", "k", "v")}
    if cfg.backward:
        out["do"] = make_activation(cfg, "do", device, extra)
    out["bias"] = make_bias_table(cfg, device, extra)
    return out


def small_config(name: str, B: int, H: int, W: int, heads: int, head_dim: int, window: int,
                 shift_h: int, shift_w: int, periodic_h: int = 0, periodic_w: int = 1,
                 index: int = 9) -> SwinConfig:
    """Ad-hoc configuration for edge-case tests."""
    return SwinConfig(name, B, H, W, heads, head_dim, window, shift_h, shift_w,
                      periodic_h, periodic_w, True, index)
