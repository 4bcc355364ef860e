"""Seeded synthetic inputs for the TSR-Adam hot path.

This module holds the workload shapes (the five benchmark configurations) and
the random-input recipes only.  It contains none of the method's arithmetic and
imports neither the CUDA library nor the CPU oracle; both sides are fed from
here with identical bits.

Gradient recipe (stands in for LLaMA pre-training gradients, which need a
dataset and a training run): low rank plus noise,
    G = sum_{i=1..s} (1/i) a_i b_i^T + noise_std * Z,
a_i in R^m, b_i in R^n, Z iid N(0,1), s = 64 signal directions, generated in
FP32 and rounded once (round-to-nearest-even) when a BF16 gradient is asked
for.  Every (config, block, step, role) gets its own seed, so each step sees a
full redraw.  Weights are 0.02 * N(0,1) in FP32.  The sketch matrix Omega is
iid N(0,1), n x (r+p), FP32.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass
from typing import List, Optional

import torch

BASE_SEED = 20260208
SIGNAL_RANK = 64
NOISE_STD = 1e-3
WEIGHT_STD = 0.02

ROLE_GRAD, ROLE_WEIGHT, ROLE_OMEGA, ROLE_INIT_GRAD, ROLE_INIT_OMEGA = 0, 1, 2, 3, 4


@dataclass(frozen=True)
class BlockShape:
    name: str
    m: int
    n: int
    r: int
    p: int
    q: int
    K: int
    is_embedding: bool = False


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    g_dtype: str          # "f32" or "bf16"
    steps: int
    blocks: tuple


def _llama(name, cid, layers, hidden, ffn, vocab, r, r_emb, p, q, K, steps) -> Workload:
    blocks: List[BlockShape] = []
    for layer in range(layers):
        for proj in ("q", "k", "v", "o"):
            blocks.append(BlockShape("l%d.%s" % (layer, proj), hidden, hidden, r, p, q, K))
        blocks.append(BlockShape("l%d.gate" % layer, ffn, hidden, r, p, q, K))
        blocks.append(BlockShape("l%d.up" % layer, ffn, hidden, r, p, q, K))
        blocks.append(BlockShape("l%d.down" % layer, hidden, ffn, r, p, q, K))
    blocks.append(BlockShape("embed", vocab, hidden, r_emb, p, q, K, True))
    return Workload(name, cid, "bf16", steps, tuple(blocks))


def workload(config_id: int) -> Workload:
    """The five benchmark configurations (config_id 0..4)."""
    if config_id == 0:
        return Workload("single-512x1376-r128-f32", 0, "f32", 10,
                        (BlockShape("single", 512, 1376, 128, 8, 1, 0),))
    if config_id == 1:
        return _llama("llama60m-r128-e64", 1, 8, 512, 1376, 32000, 128, 64, 8, 1, 100, 200)
    if config_id == 2:
        return _llama("llama130m-r256-e128", 2, 12, 768, 2048, 32000, 256, 128, 8, 1, 100, 200)
    if config_id == 3:
        return _llama("llama350m-r256-e128", 3, 24, 1024, 2736, 32000, 256, 128, 8, 1, 100, 100)
    if config_id == 4:
        return _llama("llama1b-r512-e256", 4, 24, 2048, 5461, 32000, 512, 256, 16, 2, 50, 50)
    raise ValueError("config_id must be 0..4")


def padded_ld(cols: int, elem_bytes: int) -> int:
    """Smallest leading dimension >= cols whose row pitch is a multiple of 16 bytes."""
    per = 16 // elem_bytes
    return (cols + per - 1) // per * per


def seed_for(config_id: int, block: int, step: int, role: int, base: int = BASE_SEED) -> int:
    h = hashlib.sha256(("%d/%d/%d/%d/%d" % (base, config_id, block, step, role)).encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 62) - 1)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def gradient(m: int, n: int, seed: int, dtype: torch.dtype = torch.float32, device="cpu",
             signal_rank: int = SIGNAL_RANK, noise_std: float = NOISE_STD,
             ld: Optional[int] = None) -> torch.Tensor:
    """Low-rank-plus-noise gradient, m x n view of an m x ld buffer (ld >= n, padding zeroed)."""
    gen = _gen(seed, device)
    a = torch.randn(m, signal_rank, generator=gen, device=device, dtype=torch.float32)
    b = torch.randn(n, signal_rank, generator=gen, device=device, dtype=torch.float32)
    sig = 1.0 / torch.arange(1, signal_rank + 1, device=device, dtype=torch.float32)
    g = (a * sig) @ b.t()
    if noise_std != 0.0:
        g = g + noise_std * torch.randn(m, n, generator=gen, device=device, dtype=torch.float32)
    ld = n if ld is None else ld
    buf = torch.zeros(m, ld, device=device, dtype=dtype)
    buf[:, :n] = g.to(dtype)
    return buf[:, :n]


def weights(m: int, n: int, seed: int, device="cpu", ld: Optional[int] = None) -> torch.Tensor:
    gen = _gen(seed, device)
    ld = n if ld is None else ld
    buf = torch.zeros(m, ld, device=device, dtype=torch.float32)
    buf[:, :n] = WEIGHT_STD * torch.randn(m, n, generator=gen, device=device, dtype=torch.float32)
    return buf[:, :n]


def omega(n: int, k: int, seed: int, device="cpu") -> torch.Tensor:
    return torch.randn(n, k, generator=_gen(seed, device), device=device, dtype=torch.float32)


def orthonormal(m: int, r: int, seed: int, device="cpu") -> torch.Tensor:
    """A random m x r matrix with orthonormal columns (FP32), for tests that need given bases."""
    x = torch.randn(m, r, generator=_gen(seed, "cpu"), dtype=torch.float64)
    qmat, _ = torch.linalg.qr(x)
    return qmat.to(torch.float32).to(device).contiguous()
