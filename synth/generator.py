"""Seeded synthetic inputs for the hybrid decode-attention path.

This module serves both the CUDA path and the CPU oracle and contains none of
the method's arithmetic: it only draws N(0,1) tensors from seeded torch
generators and plants the sink+recent bias that makes some layers "lazy".
The oracle never regenerates anything; tests copy back the exact bits of the
slices they check.

Recipe (per layer l, seed = BASE_SEED mixed with a tensor id and l):
  Q_tail [B, Hq, T, D], K [B, Hkv, n, D], V [B, Hkv, n, D]  ~ N(0, 1) i.i.d.
  planted layers: for each (b, kv head) u = unit vector of the mean of that
  head group's tail queries (over t and the G query heads);
  K[p] += alpha * u for p < n_sink and for p >= n - n_recent; then round to the
  storage dtype.  Decode-step q, k_new, v_new ~ N(0, 1).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

__all__ = ["BASE_SEED", "Config", "CONFIGS", "planted_layers", "make_layer", "decode_inputs", "torch_dtype"]

BASE_SEED = 241013846


@dataclass(frozen=True)
class Config:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    batch: int
    n_ctx: int          # prompt length
    n_sink: int
    n_recent: int
    w_last: int
    n_lazy: int
    dtype: str          # "f32" or "bf16"
    steps: int          # decode steps after the prompt
    alpha: float = 4.0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def capacity(self) -> int:
        return self.n_ctx + self.steps

    def scaled(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    # 1: toy stack, every element checked
    "toy": Config("toy", 2, 4, 2, 64, 1, 512, 4, 60, 16, 1, "f32", 1),
    # 2: Llama-3-8B-shaped, 32K context (the target configuration)
    "llama3_8b_32k": Config("llama3_8b_32k", 32, 32, 8, 128, 8, 32768, 4, 2044, 64, 16, "bf16", 128),
    # 3: Llama-2-7B-shaped MHA, 4K context
    "llama2_7b_4k": Config("llama2_7b_4k", 32, 32, 32, 128, 32, 4096, 4, 1020, 64, 16, "bf16", 128),
    # 4: QwQ-32B-shaped long generation (GQA group 5), ring wraps several times
    "qwq32b_longgen": Config("qwq32b_longgen", 64, 40, 8, 128, 4, 1024, 4, 4092, 64, 32, "bf16", 16384),
    # 5: Llama-3.1-8B-shaped, 128K context
    "llama31_8b_128k": Config("llama31_8b_128k", 32, 32, 8, 128, 2, 131072, 4, 4092, 64, 16, "bf16", 128),
    # 6: Llama-3-70B-shaped (80 layers, GQA group 8), 16K context
    "llama3_70b_16k": Config("llama3_70b_16k", 80, 64, 8, 128, 2, 16384, 4, 2044, 64, 40, "bf16", 128),
}


def torch_dtype(cfg: Config):
    return torch.float32 if cfg.dtype == "f32" else torch.bfloat16


def _seed(*parts: int) -> int:
    x = BASE_SEED
    for p in parts:
        x = (x * 6364136223846793005 + 1442695040888963407 + int(p)) % (1 << 63)
    return x


def planted_layers(cfg: Config, seed: int = 0):
    """Sorted list of the n_lazy planted layers: a seeded random subset (the toy
    stack plants layer 1)."""
    if cfg.name == "toy":
        return [1]
    g = torch.Generator().manual_seed(_seed(7, seed))
    perm = torch.randperm(cfg.n_layers, generator=g).tolist()
    return sorted(perm[: cfg.n_lazy])


def make_layer(cfg: Config, layer: int, planted: bool, device, capacity: int | None = None, seed: int = 0):
    """Prompt tensors of one layer: (Q_tail [B,Hq,T,D], K [B,Hkv,cap,D], V [B,Hkv,cap,D]).
    Rows >= n_ctx of K and V are zero."""
    dt = torch_dtype(cfg)
    cap = cfg.capacity if capacity is None else capacity
    B, Hq, Hkv, D, n, T = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_ctx, cfg.w_last
    g = torch.Generator(device=device).manual_seed(_seed(1, layer, seed))
    q_tail = torch.randn((B, Hq, T, D), generator=g, device=device, dtype=torch.float32).to(dt)
    K = torch.zeros((B, Hkv, cap, D), device=device, dtype=dt)
    V = torch.zeros((B, Hkv, cap, D), device=device, dtype=dt)
    K[:, :, :n].copy_(torch.randn((B, Hkv, n, D), generator=g, device=device, dtype=dt))
    V[:, :, :n].copy_(torch.randn((B, Hkv, n, D), generator=g, device=device, dtype=dt))
    if planted:
        G = cfg.group
        qm = q_tail.float().reshape(B, Hkv, G * T, D).mean(dim=2)            # [B,Hkv,D]
        u = qm / qm.norm(dim=-1, keepdim=True)
        bump = (cfg.alpha * u)[:, :, None, :]
        S, R = cfg.n_sink, cfg.n_recent
        lo = max(n - R, 0)
        if S > 0:
            K[:, :, : min(S, n)] = (K[:, :, : min(S, n)].float() + bump).to(dt)
        start = max(lo, min(S, n))                                             # no double bump on an overlap
        K[:, :, start:n] = (K[:, :, start:n].float() + bump).to(dt)
    return q_tail, K, V


def decode_inputs(cfg: Config, step: int, device, seed: int = 0):
    """(q [L,B,Hq,D], k_new [L,B,Hkv,D], v_new [L,B,Hkv,D]) of one decode step."""
    dt = torch_dtype(cfg)
    L, B, Hq, Hkv, D = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    g = torch.Generator(device=device).manual_seed(_seed(2, step, seed))
    q = torch.randn((L, B, Hq, D), generator=g, device=device, dtype=torch.float32).to(dt)
    k = torch.randn((L, B, Hkv, D), generator=g, device=device, dtype=torch.float32).to(dt)
    v = torch.randn((L, B, Hkv, D), generator=g, device=device, dtype=torch.float32).to(dt)
    return q, k, v
