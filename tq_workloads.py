"""Seeded synthetic inputs for the five evaluation configurations.

This module draws data only: it holds none of the quantiser's arithmetic and
is the single piece of code that both the CPU oracle's tests and the CUDA
path's tests/benchmark may share.  Everything is generated with torch's seeded
generators on the requested device, in row chunks, so a full 10^6 x 3072 set
can be produced directly in GPU memory.

The real datasets the paper measures on (GloVe-200, DBpedia OpenAI3 1536/3072
embeddings, Llama KV tensors) are not available; these laws stand in for
them:
  c1  d=128   i.i.d. N(0,1), unit-normalised
  c2  d=200   x_j = g_j * j^-0.3, unit-normalised
  c3  KV      K,V [heads, tokens, 128] N(0,1), 8 seeded channels per head x10, bf16
  c4  d=1536  w = g * j^-0.5; w/||w|| + mu (||mu|| = 0.3); unit-normalised
  c5  d=3072  same as c4 with j^-0.4
"""
from __future__ import annotations

import dataclasses

import torch


@dataclasses.dataclass(frozen=True)
class VectorConfig:
    name: str
    d: int
    n: int
    nq: int
    decay: float          # lambda_j = j^-decay (0 = isotropic)
    offset_norm: float    # norm of the shared mean offset (0 = none)
    data_seed: int
    query_seed: int
    pi_seed: int
    s_seed: int


CONFIGS = {
    "c1": VectorConfig("c1", 128, 4096, 64, 0.0, 0.0, 0, 1001, 52, 53),
    "c2": VectorConfig("c2", 200, 1_000_000, 10_000, 0.3, 0.0, 2, 1002, 62, 63),
    "c4": VectorConfig("c4", 1536, 1_000_000, 10_000, 0.5, 0.3, 4, 1004, 82, 83),
    "c5": VectorConfig("c5", 3072, 1_000_000, 10_000, 0.4, 0.3, 5, 1005, 92, 93),
}


def _offset_direction(cfg: VectorConfig, device) -> torch.Tensor:
    g = torch.Generator(device="cpu").manual_seed(cfg.data_seed * 7919 + 17)
    mu = torch.randn(cfg.d, generator=g, dtype=torch.float64)
    mu = mu / mu.norm() * cfg.offset_norm
    return mu.to(device=device, dtype=torch.float32)


def make_vectors(cfg: VectorConfig, count: int, seed: int, device="cpu", chunk: int = 65536,
                 out: torch.Tensor | None = None) -> torch.Tensor:
    """`count` fp32 rows from cfg's law.  Row r depends only on (seed, chunk of r)."""
    device = torch.device(device)
    if out is None:
        out = torch.empty((count, cfg.d), dtype=torch.float32, device=device)
    lam = torch.arange(1, cfg.d + 1, dtype=torch.float32, device=device).pow(-cfg.decay)
    mu = _offset_direction(cfg, device) if cfg.offset_norm > 0 else None
    for ci, start in enumerate(range(0, count, chunk)):
        rows = min(chunk, count - start)
        g = torch.Generator(device=device).manual_seed(seed * 1_000_003 + ci)
        w = torch.randn((rows, cfg.d), generator=g, dtype=torch.float32, device=device)
        w.mul_(lam)
        w.div_(w.norm(dim=1, keepdim=True))
        if mu is not None:
            w.add_(mu)
            w.div_(w.norm(dim=1, keepdim=True))
        out[start:start + rows] = w
    return out


def database(cfg: VectorConfig, count: int | None = None, device="cpu") -> torch.Tensor:
    return make_vectors(cfg, cfg.n if count is None else count, cfg.data_seed, device)


def queries(cfg: VectorConfig, count: int | None = None, device="cpu") -> torch.Tensor:
    return make_vectors(cfg, cfg.nq if count is None else count, cfg.query_seed, device)


def kv_cache(heads: int = 8, tokens: int = 32768, head_dim: int = 128, q_per_kv: int = 4,
             seed: int = 3, outlier_seed: int = 7, device="cpu"):
    """Config c3: (K, V, Q) = bf16 [heads, tokens, head_dim] x2 and bf16
    [heads*q_per_kv, head_dim]; 8 seeded channels per KV head are scaled x10
    in both K and V."""
    device = torch.device(device)
    g = torch.Generator(device=device).manual_seed(seed)
    K = torch.randn((heads, tokens, head_dim), generator=g, dtype=torch.float32, device=device)
    V = torch.randn((heads, tokens, head_dim), generator=g, dtype=torch.float32, device=device)
    Q = torch.randn((heads * q_per_kv, head_dim), generator=g, dtype=torch.float32, device=device)
    go = torch.Generator(device="cpu").manual_seed(outlier_seed)
    for h in range(heads):
        ch = torch.randperm(head_dim, generator=go)[:8].to(device)
        K[h][:, ch] *= 10.0
        V[h][:, ch] *= 10.0
    return K.to(torch.bfloat16), V.to(torch.bfloat16), Q.to(torch.bfloat16)
