"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors.  It holds none of the method's arithmetic (no scoring,
no selection, no product) and is the one module that both the tests of the CPU oracle and the
CUDA path may share.

Conventions: one torch.Generator per tensor, seeded  seed (A / Q), seed+1 (B / K), seed+2 (V),
seed+3 (choice of special columns); fp32 draw, then round-to-nearest-even to bf16.
"""
from __future__ import annotations

import math
from typing import Tuple

import torch


def _gen(seed: int, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gaussian(shape, std: float, seed: int, dtype=torch.bfloat16, device: str = "cpu") -> torch.Tensor:
    x = torch.randn(*shape, generator=_gen(seed, device), dtype=torch.float32, device=device)
    if std != 1.0:
        x *= std
    return x.to(dtype)


def outlier_product(M: int = 64, K: int = 512, N: int = 256, n_outlier: int = 8, gain: float = 20.0,
                    seed: int = 0, dtype=torch.bfloat16) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Single product with outlier channels: A ~ N(0,1) with n_outlier random columns scaled by
    gain, B ~ N(0, 1/K).  Returns (A [M,K], B [K,N], outlier column indices)."""
    A = torch.randn(M, K, generator=_gen(seed), dtype=torch.float32)
    cols = torch.randperm(K, generator=_gen(seed + 3))[:n_outlier]
    A[:, cols] *= gain
    B = torch.randn(K, N, generator=_gen(seed + 1), dtype=torch.float32) / math.sqrt(K)
    return A.to(dtype), B.to(dtype), cols


def heavy_tailed_activations(M: int, K: int, seed: int = 0, frac: float = 0.01, nu: int = 3,
                             dtype=torch.bfloat16, device: str = "cpu") -> torch.Tensor:
    """Activations ~ N(0,1) in which ceil(frac*K) randomly chosen channels (columns) have
    i.i.d. Student-t(nu) entries, drawn as z / sqrt(chi2_nu / nu)."""
    g = _gen(seed, device)
    A = torch.randn(M, K, generator=g, dtype=torch.float32, device=device)
    n_heavy = int(math.ceil(frac * K)) if frac > 0 else 0
    if n_heavy > 0:
        cols = torch.randperm(K, generator=_gen(seed + 3))[:n_heavy].to(device)
        z = torch.randn(M, n_heavy, generator=g, dtype=torch.float32, device=device)
        chi2 = torch.randn(M, n_heavy, nu, generator=g, dtype=torch.float32, device=device).square_().sum(-1)
        A[:, cols] = z / torch.sqrt(chi2 / nu)
    return A.to(dtype)


def weight(K: int, N: int, seed: int = 1, std: float = 0.02, dtype=torch.bfloat16,
           device: str = "cpu") -> torch.Tensor:
    """Projection weight stored K x N (contraction slices contiguous), ~ N(0, std^2)."""
    return gaussian((K, N), std, seed, dtype, device)


def mlp_product(M: int, K: int, N: int, seed: int = 0, dtype=torch.bfloat16, device: str = "cpu"):
    """MLP / linear projection workload: heavy-tailed activations and a N(0, 0.02^2) weight."""
    return heavy_tailed_activations(M, K, seed, dtype=dtype, device=device), weight(K, N, seed + 1, dtype=dtype,
                                                                                    device=device)


def attention_qkv(B: int, Hq: int, Hkv: int, Lq: int, Lk: int, Dh: int, seed: int = 0, n_outlier: int = 4,
                  gain: float = 10.0, dtype=torch.bfloat16, device: str = "cpu"):
    """Q [B,Hq,Lq,Dh], K,V [B,Hkv,Lk,Dh] ~ N(0,1).  Per query head, n_outlier feature dims
    (seeded) are scaled by gain in Q, and the same dims in the kv head it reads are scaled in K."""
    Q = torch.randn(B, Hq, Lq, Dh, generator=_gen(seed, device), dtype=torch.float32, device=device)
    K = torch.randn(B, Hkv, Lk, Dh, generator=_gen(seed + 1, device), dtype=torch.float32, device=device)
    V = torch.randn(B, Hkv, Lk, Dh, generator=_gen(seed + 2, device), dtype=torch.float32, device=device)
    if n_outlier > 0:
        g = _gen(seed + 3)
        group = Hq // Hkv
        for h in range(Hkv):
            dims = torch.randperm(Dh, generator=g)[:n_outlier].to(device)
            K[:, h, :, dims] *= gain
            Q[:, h * group:(h + 1) * group, :, dims] *= gain
    return Q.to(dtype), K.to(dtype), V.to(dtype)


def attention_probs(L: int, H: int, Dh: int = 128, seed: int = 0, causal: bool = True,
                    device: str = "cpu") -> torch.Tensor:
    """A materialised attention-weight input P [H, L, L] bf16 for the PV product taken on its own:
    P = bf16(softmax_fp32(mask(Q K^T / sqrt(Dh)))) with Q, K ~ N(0,1) bf16, built head by head."""
    P = torch.empty(H, L, L, dtype=torch.bfloat16, device=device)
    for h in range(H):
        q = gaussian((L, Dh), 1.0, seed + 10 * h, torch.bfloat16, device).float()
        k = gaussian((L, Dh), 1.0, seed + 10 * h + 1, torch.bfloat16, device).float()
        s = (q @ k.T) / math.sqrt(Dh)
        if causal:
            s = s.masked_fill(torch.ones(L, L, dtype=torch.bool, device=device).triu(1), float("-inf"))
        P[h] = torch.softmax(s, dim=-1).to(torch.bfloat16)
    return P
