"""Seeded synthetic inputs for the QAQ hot path (KV caches, queries, score windows).

This module only draws random numbers with the shapes and value structure of
LLaMA-2-like KV caches (stand-ins for the caches the paper measured on public
evaluation suites, Section 5.1); it contains none of the method's arithmetic and
is the one module the tests feed to both the CUDA path and the CPU checker.

Recipe (per layer, generator seeded with ``seed + layer``):
  * K, V [B,H,T,D] fp16:  x = s_c * z,  z ~ N(0,1) or Student-t(nu=3),
    s_c ~ lognormal(0, 0.5) per (head, channel, tensor) (or 1),
    a fraction ``outlier_frac`` of entries replaced by  +-u * s_c,
    u ~ U[outlier_lo, outlier_hi];
  * q [B,H,D] fp16 ~ N(0,1);
  * score window ring [B,H,W,T] fp32: rows of a probability vector over the T
    tokens that persists from row to row (shared per-token base logits ~ N(0,1.3^2)
    plus N(0,0.3^2) row noise) with rare +4 jumps on single rows, the "exceptions"
    of Section 3.2; nvalid [B,H,T] u8 = number of valid rows per token.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    heads: int
    head_dim: int
    tokens: int
    window: int
    alpha: float            # outlier proportion handed to the method (both tails)
    bits_min: int = 2
    bits_max: int = 8
    layers: int = 1
    dist: str = "normal"    # "normal" | "student3"
    channel_scales: bool = True
    outlier_frac: float = 0.01
    outlier_lo: float = 10.0
    outlier_hi: float = 20.0
    seed: int = 0
    grow_to: int = 0        # streaming: tokens appended one by one up to this length

    @property
    def bh(self) -> int:
        return self.batch * self.heads


CONFIGS = {
    # tiny single layer
    "C1": Workload("C1-tiny", 1, 4, 64, 512, 5, 0.01, outlier_lo=15.0, outlier_hi=15.0, seed=0),
    # LLaMA-7B-shaped single layer
    "C2": Workload("C2-7B-layer", 1, 32, 128, 4096, 32, 0.01, seed=1),
    # LLaMA-7B-shaped full cache
    "C3": Workload("C3-7B-full", 8, 32, 128, 4096, 32, 0.01, layers=32, seed=1000),
    # LLaMA-13B-shaped cache, heavy tails
    "C4": Workload("C4-13B-heavy", 4, 40, 128, 8192, 64, 0.05, layers=40, dist="student3",
                   outlier_frac=0.05, seed=2000),
    # long-context streaming decode
    "C5": Workload("C5-stream", 1, 32, 128, 32768, 32, 0.01, channel_scales=False, seed=3, grow_to=131072),
}


def scaled(wl: Workload, **kw) -> Workload:
    """A copy of a workload with some fields changed (smaller test-sized variants)."""
    return replace(wl, **kw)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_kv(wl: Workload, layer: int = 0, device="cpu", tokens: int | None = None):
    """K, V as fp16 tensors [B,H,T,D]."""
    T = wl.tokens if tokens is None else tokens
    g = _gen(device, wl.seed + layer)
    out = []
    for _ in range(2):
        shape = (wl.batch, wl.heads, T, wl.head_dim)
        z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        if wl.dist == "student3":
            chi = torch.zeros(shape, device=device, dtype=torch.float32)
            for _k in range(3):
                chi += torch.randn(shape, generator=g, device=device, dtype=torch.float32) ** 2
            z = z / torch.sqrt(chi / 3.0)
        if wl.channel_scales:
            s = torch.exp(0.5 * torch.randn((1, wl.heads, 1, wl.head_dim), generator=g, device=device))
        else:
            s = torch.ones((1, wl.heads, 1, wl.head_dim), device=device)
        x = z * s
        if wl.outlier_frac > 0:
            m = torch.rand(shape, generator=g, device=device) < wl.outlier_frac
            u = wl.outlier_lo + (wl.outlier_hi - wl.outlier_lo) * torch.rand(shape, generator=g, device=device)
            sign = torch.where(torch.rand(shape, generator=g, device=device) < 0.5, -1.0, 1.0)
            x = torch.where(m, sign * u * s, x)
        out.append(x.clamp_(-60000.0, 60000.0).to(torch.float16).contiguous())
    return out[0], out[1]


def make_query(wl: Workload, layer: int = 0, step: int = 0, device="cpu"):
    """One decode query per (b,h): fp16 [B,H,D]."""
    g = _gen(device, (wl.seed + layer) * 7919 + 17 + step)
    q = torch.randn((wl.batch, wl.heads, wl.head_dim), generator=g, device=device, dtype=torch.float32)
    return q.to(torch.float16).contiguous()


def make_score_ring(wl: Workload, layer: int = 0, device="cpu", tokens: int | None = None, ragged: bool = False):
    """ring fp32 [B,H,W,T] and nvalid u8 [B,H,T]."""
    T = wl.tokens if tokens is None else tokens
    W = wl.window
    g = _gen(device, (wl.seed + layer) * 104729 + 5)
    base = 1.3 * torch.randn((wl.batch, wl.heads, 1, T), generator=g, device=device, dtype=torch.float64)
    noise = 0.3 * torch.randn((wl.batch, wl.heads, W, T), generator=g, device=device, dtype=torch.float64)
    jump = (torch.rand((wl.batch, wl.heads, W, T), generator=g, device=device) < 0.002).to(torch.float64) * 4.0
    logits = base + noise + jump
    ring = torch.softmax(logits, dim=-1).to(torch.float32).contiguous()
    if ragged:
        nvalid = torch.randint(0, W + 1, (wl.batch, wl.heads, T), generator=g, device=device).to(torch.uint8)
    else:
        nvalid = torch.full((wl.batch, wl.heads, T), W, device=device, dtype=torch.uint8)
    return ring, nvalid.contiguous()
