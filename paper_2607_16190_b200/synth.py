"""Seeded synthetic Q/K/V for the benchmark configurations.

This module holds none of the method's arithmetic: it only draws inputs.  Both the
CUDA path and the CPU oracle are fed the bf16 tensors it returns.

Recipe (stands in for real video-DiT activations, which need model weights):
  per layer seed:  omega_m ~ N(0, 3^2 I_3), phi_m ~ U[0, 2 pi), m < F
  per token (t,y,x): u = (t/T, y/Y, x/X);  f_m = cos(omega_m . u + phi_m)
  per head:        Wq, Wk ~ N(0, 1/16) of shape F x d;  temperature s_h
                   Q = s_h (f Wq + 0.5 eps),  K = f Wk + 0.5 eps',  V ~ N(0, 1)
  rounded once to bf16, returned as [1, N, H, d] with N in raster order over (T, Y, X).
Head temperatures: log-uniform on [0.5, 4], or heavy-tailed exp(N(0.5, 0.8^2)) clipped to
[0.3, 8] (spreads retained-block counts across heads by more than an order of magnitude).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Config:
    name: str
    H: int
    d: int
    grid: tuple          # (T, Y, X)
    tile: tuple          # (tT, tY, tX)
    p: float
    k_floor: int
    features: int
    temperature: str     # "loguniform" | "heavytail"
    seed: int = 0

    @property
    def tokens(self) -> int:
        return self.grid[0] * self.grid[1] * self.grid[2]

    @property
    def block_tokens(self) -> int:
        return self.tile[0] * self.tile[1] * self.tile[2]

    @property
    def num_blocks(self) -> int:
        return math.prod(-(-g // t) for g, t in zip(self.grid, self.tile))

    @property
    def sm_scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    def with_(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    "tiny": Config("tiny", 2, 64, (4, 8, 8), (1, 8, 8), 0.9, 1, 16, "loguniform", seed=1),
    "small": Config("small", 12, 128, (8, 16, 16), (2, 8, 8), 0.9, 2, 32, "loguniform", seed=2),
    "wan480p": Config("wan480p", 40, 128, (21, 30, 52), (1, 8, 16), 0.9, 4, 64, "loguniform", seed=3),
    "wan720p": Config("wan720p", 40, 128, (21, 45, 80), (1, 8, 16), 0.9, 4, 64, "heavytail", seed=4),
}
SWEEP_P = (0.5, 0.7, 0.9, 0.95, 0.99)
SWEEP_LAYERS = 40


def sweep_layer(layer: int) -> Config:
    """Config of one layer of the 720p sweep (distinct seed per layer)."""
    return CONFIGS["wan720p"].with_(name=f"wan720p_layer{layer}", seed=1000 + layer)


def head_temperatures(cfg: Config, gen: torch.Generator) -> torch.Tensor:
    if cfg.temperature == "loguniform":
        u = torch.rand(cfg.H, generator=gen, dtype=torch.float64)
        return torch.exp(math.log(0.5) + u * (math.log(4.0) - math.log(0.5)))
    if cfg.temperature == "heavytail":
        z = torch.randn(cfg.H, generator=gen, dtype=torch.float64)
        return torch.exp(0.5 + 0.8 * z).clamp(0.3, 8.0)
    raise ValueError(cfg.temperature)


def make_qkv(cfg: Config, device: str | torch.device = "cpu"):
    """Return (q, k, v), each [1, N, H, d] bf16 on ``device``, plus the head temperatures.

    Small parameters are drawn on the CPU (identical on every device); the per-token noise
    is drawn with a seeded generator on ``device``.
    """
    device = torch.device(device)
    T, Y, X = cfg.grid
    N, H, d, F = cfg.tokens, cfg.H, cfg.d, cfg.features
    cg = torch.Generator(device="cpu").manual_seed(cfg.seed)
    omega = 3.0 * torch.randn(F, 3, generator=cg, dtype=torch.float64)
    phi = 2.0 * math.pi * torch.rand(F, generator=cg, dtype=torch.float64)
    s_h = head_temperatures(cfg, cg)
    wq = 0.25 * torch.randn(H, F, d, generator=cg, dtype=torch.float64)
    wk = 0.25 * torch.randn(H, F, d, generator=cg, dtype=torch.float64)

    t = torch.arange(T, dtype=torch.float64) / T
    y = torch.arange(Y, dtype=torch.float64) / Y
    x = torch.arange(X, dtype=torch.float64) / X
    u = torch.stack(torch.meshgrid(t, y, x, indexing="ij"), dim=-1).reshape(N, 3)
    feat = torch.cos(u @ omega.T + phi).to(torch.float32).to(device)   # [N, F]

    dg = torch.Generator(device=device).manual_seed(cfg.seed + 7919)
    q = torch.empty(1, N, H, d, dtype=torch.bfloat16, device=device)
    k = torch.empty_like(q)
    v = torch.empty_like(q)
    for h in range(H):
        wqh = wq[h].to(torch.float32).to(device)
        wkh = wk[h].to(torch.float32).to(device)
        eq = torch.randn(N, d, generator=dg, dtype=torch.float32, device=device)
        ek = torch.randn(N, d, generator=dg, dtype=torch.float32, device=device)
        ev = torch.randn(N, d, generator=dg, dtype=torch.float32, device=device)
        q[0, :, h] = (float(s_h[h]) * (feat @ wqh + 0.5 * eq)).to(torch.bfloat16)
        k[0, :, h] = (feat @ wkh + 0.5 * ek).to(torch.bfloat16)
        v[0, :, h] = ev.to(torch.bfloat16)
    return q, k, v, s_h


def bf16_bits(x: torch.Tensor):
    """Host numpy uint16 view of a bf16 tensor's bit patterns (what the oracle takes)."""
    import numpy as np

    return x.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a, device: str | torch.device = "cpu") -> torch.Tensor:
    import numpy as np

    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)
