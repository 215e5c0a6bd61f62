"""Seeded synthetic inputs for the compression pass.

This module only *draws inputs*: post-RoPE window queries and a prefilled K/V
cache with the qualitative structure of real long-context attention (a few
attention-sink tokens at the start, a sparse set of heavy-hitter tokens).  It
contains none of the method's arithmetic and is the one module that both the
CUDA path's tests/benchmarks and the CPU oracle's tests consume, so that both
sides see bit-identical tensors.

The shapes follow the models the paper evaluates (LLaMA-3.1-8B: 32 layers,
32 query heads, 8 KV heads, head_dim 128; a GQA-4 long-context shape); the
values stand in for real prompts, which are not available offline.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import torch


@dataclasses.dataclass(frozen=True)
class WorkloadConfig:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_ctx: int
    window: int
    batch: int = 1
    dtype: str = "bf16"            # "bf16" | "f32"
    retention: float = 0.25        # rho = 1 - r_target
    n_sinks: int = 4
    hh_frac: float = 0.01          # heavy-hitter density
    hh_mode: str = "uniform"       # "uniform" | "bursts" | "loguniform" | "ties"
    hh_layer_strength: bool = True  # alpha_l ~ U(0.5, 3) per layer, else 1
    elem_std: Optional[float] = None  # std of the base normal draw; None -> 1/sqrt(head_dim)
    seed: int = 0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def budget(self) -> int:
        """B_total = floor(rho * L * N) token slots per sequence."""
        return int(math.floor(self.retention * self.n_layers * self.n_ctx + 1e-9))

    def replace(self, **kw) -> "WorkloadConfig":
        return dataclasses.replace(self, **kw)


# The benchmark configurations (names are stable identifiers used by bench.py and the tests).
TINY = WorkloadConfig("tiny", 2, 4, 2, 64, 512, 16, dtype="f32", retention=0.25, hh_frac=0.02,
                      hh_layer_strength=False)
LLAMA8B_8K = WorkloadConfig("llama8b_8k", 32, 32, 8, 128, 8192, 32, retention=0.20, hh_frac=0.01)
LLAMA8B_32K = WorkloadConfig("llama8b_32k", 32, 32, 8, 128, 32768, 32, retention=0.25,
                             hh_frac=0.005, hh_mode="bursts")
GQA4_128K = WorkloadConfig("gqa4_128k", 28, 28, 4, 128, 131072, 64, retention=0.10, hh_frac=0.01,
                           hh_mode="loguniform")
TIES_4K = WorkloadConfig("ties_4k", 32, 32, 8, 128, 4096, 32, retention=0.25, hh_frac=0.01,
                         hh_mode="ties")

CONFIGS = {c.name: c for c in (TINY, LLAMA8B_8K, LLAMA8B_32K, GQA4_128K, TIES_4K)}


def sweep_config(n_ctx: int, batch: int, retention: float) -> WorkloadConfig:
    """A point of the 8B-shape sweep (N x batch x retention)."""
    return LLAMA8B_8K.replace(name="llama8b_n%d_b%d_r%02d" % (n_ctx, batch, round(retention * 100)),
                              n_ctx=n_ctx, batch=batch, retention=retention)


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[name]


@dataclasses.dataclass
class Workload:
    cfg: WorkloadConfig
    q: List[torch.Tensor]   # L x [Bt, Hq, w, d]
    k: List[torch.Tensor]   # L x [Bt, Hkv, N, d]
    v: List[torch.Tensor]   # L x [Bt, Hkv, N, d]

    def to(self, device) -> "Workload":
        return Workload(self.cfg, [t.to(device) for t in self.q], [t.to(device) for t in self.k],
                        [t.to(device) for t in self.v])

    def bytes_kv(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.k + self.v)


def _hh_positions(cfg: WorkloadConfig, gen: torch.Generator, device) -> torch.Tensor:
    """Heavy-hitter positions for one (layer, sequence, head); never a sink position."""
    N, s = cfg.n_ctx, cfg.n_sinks
    if cfg.hh_mode == "uniform":
        n = int(math.floor(cfg.hh_frac * N))
        perm = torch.randperm(N - s, generator=gen, device=device)[:n] + s
        return perm
    if cfg.hh_mode == "bursts":
        burst = 64
        nb = max(1, int(round(cfg.hh_frac * N / burst)))
        slots = torch.randperm(N // burst - 1, generator=gen, device=device)[:nb] + 1
        return (slots[:, None] * burst + torch.arange(burst, device=device)[None, :]).reshape(-1)
    if cfg.hh_mode == "loguniform":
        n = int(math.floor(cfg.hh_frac * N))
        u = torch.rand(n, generator=gen, device=device)
        pos = torch.exp(u * math.log(N)).floor().long().clamp_(s, N - 1)
        return torch.unique(pos)
    raise ValueError(cfg.hh_mode)


def make_layer(cfg: WorkloadConfig, gen: torch.Generator, device, alpha: float):
    """Draw (Q, K, V) of one layer: base normal draw, then sinks and heavy hitters on K."""
    Bt, Hq, Hkv, d, N, w, G = (cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_ctx,
                               cfg.window, cfg.group)
    sigma = cfg.elem_std if cfg.elem_std is not None else 1.0 / math.sqrt(d)
    f32 = torch.float32
    q = torch.randn((Bt, Hq, w, d), generator=gen, device=device, dtype=f32) * sigma
    if cfg.hh_mode == "ties":
        # every key row is one fixed vector; a sparse set of rows gets additive noise
        base = torch.randn((Bt, Hkv, 1, d), generator=gen, device=device, dtype=f32) * sigma
        k = base.expand(Bt, Hkv, N, d).clone()
        n = max(1, int(math.floor(cfg.hh_frac * N)))
        for b in range(Bt):
            for h in range(Hkv):
                pos = torch.randperm(N, generator=gen, device=device)[:n]
                k[b, h, pos] += torch.randn((n, d), generator=gen, device=device, dtype=f32) * sigma
    else:
        k = torch.randn((Bt, Hkv, N, d), generator=gen, device=device, dtype=f32) * sigma
    v = torch.randn((Bt, Hkv, N, d), generator=gen, device=device, dtype=f32) * sigma
    if cfg.hh_mode != "ties":
        # mean window query of the G query heads that share KV head h, and its direction
        qbar = q.reshape(Bt, Hkv, G * w, d).mean(dim=2)                 # [Bt, Hkv, d]
        u = qbar / qbar.norm(dim=-1, keepdim=True).clamp_min(1e-30)
        k[:, :, : cfg.n_sinks] += (3.0 * sigma) * u[:, :, None, :]
        for b in range(Bt):
            for h in range(Hkv):
                pos = _hh_positions(cfg, gen, device)
                k[b, h, pos] = (alpha * 2.0) * qbar[b, h]
    dt = torch_dtype(cfg.dtype)
    return q.to(dt), k.to(dt), v.to(dt)


def make_workload(cfg: WorkloadConfig, device="cpu", layers: Optional[range] = None) -> Workload:
    """Draw the whole workload (or the given subset of layers, identical to the full draw's)."""
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed)
    if cfg.hh_layer_strength:
        alphas = (torch.rand(cfg.n_layers, generator=gen, device=device) * 2.5 + 0.5).tolist()
    else:
        alphas = [1.0] * cfg.n_layers
    want = set(range(cfg.n_layers)) if layers is None else set(layers)
    last = max(want) if want else -1
    qs, ks, vs = [], [], []
    for l in range(cfg.n_layers):
        if l > last:
            break
        q, k, v = make_layer(cfg, gen, device, alphas[l])
        if l in want:
            qs.append(q)
            ks.append(k)
            vs.append(v)
    sub = cfg if layers is None else cfg.replace(n_layers=len(qs))
    return Workload(sub, qs, ks, vs)
