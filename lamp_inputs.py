"""Seeded synthetic inputs shaped like Qwen3 / Gemma 3 attention (shared by the oracle
tests and the CUDA tests; holds none of the method's arithmetic).

The paper evaluates on real model activations (Qwen3, Gemma 3 on C4 / MMLU / Wikitext /
ARC-Challenge); neither weights nor data are available, so these tensors stand in for
them: QK-normalised rows with per-channel gains, a few outlier channels and an
attention-sink key, which is the structure Sec. 3.3 of the paper relies on.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

OUTLIER_CHANNELS = (5, 37, 70, 101)


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    B: int
    Hq: int
    Hkv: int
    N: int
    D: int
    causal: bool = True
    window: int = 0
    qk_norm: bool = True
    scale_mults: tuple = (1.0,)
    layers: tuple = field(default_factory=lambda: (("global", 0),))


CONFIGS = {
    0: Config(0, "tiny", 1, 1, 1, 256, 128, qk_norm=False),
    1: Config(1, "qwen3-0.6b-shaped", 1, 16, 8, 2048, 128),
    2: Config(2, "qwen3-8b-shaped", 4, 32, 8, 8192, 128),
    3: Config(3, "gemma3-4b-shaped", 2, 8, 4, 8192, 256, layers=(("local", 1024), ("global", 0))),
    4: Config(4, "long-context", 1, 32, 8, 32768, 128, scale_mults=(0.5, 1.0, 2.0, 4.0, 8.0)),
}


def softmax_scale(D: int, mult: float = 1.0) -> float:
    """(float)(mult / sqrt(D)) as an fp32 value."""
    return float(torch.tensor(mult / math.sqrt(float(D)), dtype=torch.float64).to(torch.float32))


def make_qkv(cfg: Config, *, B=None, Hq=None, Hkv=None, N=None, seed=None):
    """Return (q, k, v) CPU bf16 tensors [B, H, N, D] for a config (sizes may be overridden
    to get the same value distribution at a smaller shape)."""
    B = cfg.B if B is None else B
    Hq = cfg.Hq if Hq is None else Hq
    Hkv = cfg.Hkv if Hkv is None else Hkv
    N = cfg.N if N is None else N
    D = cfg.D
    gen = torch.Generator().manual_seed(1000 + cfg.index if seed is None else seed)
    q = torch.randn(B, Hq, N, D, generator=gen, dtype=torch.float32)
    k = torch.randn(B, Hkv, N, D, generator=gen, dtype=torch.float32)
    v = torch.randn(B, Hkv, N, D, generator=gen, dtype=torch.float32)
    if cfg.qk_norm:
        gq = torch.rand(D, generator=gen) * 1.5 + 0.5
        gk = torch.rand(D, generator=gen) * 1.5 + 0.5
        for c in OUTLIER_CHANNELS:
            gq[c] *= 10.0
            gk[c] *= 10.0
        q = q * torch.rsqrt(q.pow(2).mean(-1, keepdim=True) + 1e-6) * gq
        k = k * torch.rsqrt(k.pow(2).mean(-1, keepdim=True) + 1e-6) * gk
    # attention sink: key 0 += 6 * (mean query of the query heads that read this kv head)
    qbar = q.view(B, Hkv, Hq // Hkv, N, D).mean(dim=(2, 3))
    k[:, :, 0, :] += 6.0 * qbar
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


def sample_units(cfg: Config, n: int, seed: int = 7, *, B=None, Hq=None, N=None):
    """A seeded spread of (b, h, g) units over batch, head and position; always holds the
    first and the last group."""
    B = cfg.B if B is None else B
    Hq = cfg.Hq if Hq is None else Hq
    N = cfg.N if N is None else N
    G = N // 32
    gen = torch.Generator().manual_seed(seed)
    total = B * Hq * G
    if n >= total:
        idx = torch.arange(total)
    else:
        idx = torch.randperm(total, generator=gen)[:n]
        idx[0] = total - 1
        idx[1] = 0
    b = idx // (Hq * G)
    h = (idx // G) % Hq
    g = idx % G
    return torch.stack([b, h, g], -1).to(torch.int32).numpy()
