"""Seeded synthetic inputs, shared by the CUDA tests, the oracle tests and the benchmark.

This module holds no arithmetic of the method (no layout function, no product,
no block count): it only draws numbers, rounds them to bf16 once and names the
shapes of the workloads.  The same bits are handed to the CUDA library and to
the oracle.

Shapes stand in for the matmuls the paper traces from Llama-3.1 70B (dense
projections) and Qwen-3 30B-A3B (128 experts, top-8 routing); values are random
because neither timing nor layout depends on trained weights.
"""
from __future__ import annotations

import numpy as np
import torch

BASE_SEED = 260704031

# (name, K, N): weight operands, logically K x N, N contiguous when row-major.
LLAMA70B_PROJ = (
    ("qkv", 8192, 10240),
    ("o", 8192, 8192),
    ("gate_up", 8192, 57344),
    ("down", 28672, 8192),
)
LLAMA_DECODE_M = (1, 8, 32)
LLAMA_PREFILL_M = 4096

QWEN_MOE = dict(experts=128, hidden=2048, inter=768, tokens=256, topk=8, zipf_alpha=1.1)
QWEN_MOE_PROJ = (("moe_gate_up", 2048, 1536), ("moe_down", 768, 2048))
QWEN_ATTN_PROJ = (("q", 2048, 4096), ("k", 2048, 512), ("v", 2048, 512), ("o", 4096, 2048))

DEFAULT_G = 4096
DEFAULT_BLOCK = (16, 128)        # 16 rows x 128 bf16 columns = 4 KB


def _gen(seed: int, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(BASE_SEED * 1000003 + int(seed))
    return g


def bf16_normal(shape, std: float, seed: int, device: str = "cpu") -> torch.Tensor:
    """N(0, std) in fp32, rounded once (nearest-even) to bf16."""
    x = torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return (x * std).to(torch.bfloat16)


def bf16_uniform(shape, lo: float, hi: float, seed: int, device: str = "cpu") -> torch.Tensor:
    x = torch.rand(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return (x * (hi - lo) + lo).to(torch.bfloat16)


def bf16_integers(shape, lo: int, hi: int, seed: int, device: str = "cpu") -> torch.Tensor:
    """Integer-valued bf16 in [lo, hi]: products and partial sums stay exact in fp32."""
    x = torch.randint(lo, hi + 1, shape, generator=_gen(seed, device), device=device)
    return x.to(torch.bfloat16)


def one_hot_rows(M: int, K: int, seed: int, device: str = "cpu"):
    """A with row i = unit vector e_{k_i}; returns (A bf16 [M,K], k_i int64 [M])."""
    ks = torch.randint(0, K, (M,), generator=_gen(seed, "cpu"))
    A = torch.zeros((M, K), dtype=torch.bfloat16)
    A[torch.arange(M), ks] = 1.0
    return A.to(device), ks


def random_bytes(n: int, seed: int) -> np.ndarray:
    return np.random.default_rng(BASE_SEED + seed).integers(0, 256, size=n, dtype=np.uint8)


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 numpy array of the same shape (host copy of the bit patterns)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


FP8 = torch.float8_e4m3fn


def fp8_normal(shape, std: float, seed: int, device: str = "cpu") -> torch.Tensor:
    """N(0, std) in fp32, rounded once to FP8 (E4M3)."""
    x = torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return (x * std).clamp_(-448.0, 448.0).to(FP8)


def fp8_integers(shape, lo: int, hi: int, seed: int, device: str = "cpu") -> torch.Tensor:
    """Integer-valued FP8 in [lo, hi] (|values| <= 16 are exact in E4M3)."""
    assert -16 <= lo <= hi <= 16
    x = torch.randint(lo, hi + 1, shape, generator=_gen(seed, device), device=device)
    return x.to(torch.float32).to(FP8)


def bits8(t: torch.Tensor) -> np.ndarray:
    """FP8 tensor -> uint8 numpy array of the same shape (host copy of the bit patterns)."""
    assert t.dtype == FP8
    return t.detach().contiguous().cpu().view(torch.uint8).numpy()


def zipf_topk_routing(tokens: int, experts: int, topk: int, alpha: float, seed: int):
    """Top-k routing with Zipf(alpha) expert popularity.

    Each token draws `topk` distinct experts one after another, without
    replacement, with P(rank r) proportional to r**-alpha over the ranks still
    available; ranks map to expert ids through a seeded permutation.  Returns
    (offsets int32 [experts+1], counts int64 [experts], expert_of_row int32 [tokens*topk]),
    rows sorted by expert.
    """
    rng = np.random.default_rng(BASE_SEED + 7919 * seed + 17)
    weight = np.arange(1, experts + 1, dtype=np.float64) ** (-alpha)
    rank_to_expert = rng.permutation(experts)
    counts = np.zeros(experts, dtype=np.int64)
    for _ in range(tokens):
        w = weight.copy()
        for _ in range(topk):
            r = rng.choice(experts, p=w / w.sum())
            counts[rank_to_expert[r]] += 1
            w[r] = 0.0
    offsets = np.zeros(experts + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    expert_of_row = np.repeat(np.arange(experts, dtype=np.int32), counts)
    return offsets, counts, expert_of_row
