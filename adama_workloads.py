"""Seeded synthetic inputs and workload shapes shared by the tests, the smoke
check and the benchmark.

This module holds no optimizer arithmetic: it only names shapes and draws
normally distributed tensors from a seed.  Both the fp64 CPU oracle and the
CUDA library are fed from here so that they see the same bit patterns (the
tensor is drawn once, in its storage dtype, and the oracle widens those bits
exactly to float64).

Distributions follow the workload descriptions: "N(0, s)" means standard
deviation s.  Seeds: 1000*config + 100*step + micro (+ 7919*layer for stacks).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import torch

BETA1 = 0.9
BETA2 = 0.999
EPS = 1e-8
LR = 1e-3


def seed_for(config: int, step: int = 0, micro: int = 0, layer: int = 0) -> int:
    return 1000 * config + 100 * step + micro + 7919 * layer


def normal(shape, std: float, dtype: torch.dtype, seed: int, device="cpu") -> torch.Tensor:
    """N(0, std) drawn in fp32 from `seed` on `device`, then rounded once to `dtype`.

    CPU and CUDA generators give different streams; a parity test draws on one
    device and copies the bits to the other side."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    x = torch.empty(shape, dtype=torch.float32, device=device)
    x.normal_(0.0, 1.0, generator=gen)
    x.mul_(std)
    return x if dtype == torch.float32 else x.to(dtype)


def small_integers(shape, bound: int, dtype: torch.dtype, seed: int, device="cpu") -> torch.Tensor:
    """Integer-valued tensor in [-bound, bound]; exactly representable in bf16 for
    bound <= 256, so products and short sums of them are exact in fp32."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    x = torch.randint(-bound, bound + 1, shape, generator=gen, device=device)
    return x.to(dtype)


@dataclass(frozen=True)
class FlatConfig:
    """A flat parameter buffer folded with per-micro-batch gradients."""
    config: int
    n: int
    n_micro: int
    steps: int
    grad_dtype: torch.dtype
    grad_std: float
    w_std: float = 0.02


@dataclass(frozen=True)
class LinearConfig:
    """One linear layer: X [tokens, d_in], dY [tokens, d_out], W/m/v [d_in, d_out]."""
    config: int
    tokens: int
    d_in: int
    d_out: int
    n_micro: int
    steps: int
    x_std: float = 1.0
    dy_std: float = 1e-2
    w_std: float = 0.02


# config 1: one fp32 tensor 1024x1024, fp32 gradients, N=4, 3 steps
CONFIG1 = FlatConfig(config=1, n=1024 * 1024, n_micro=4, steps=3,
                     grad_dtype=torch.float32, grad_std=1e-2)
# config 2: BERT-large-sized flat buffer, bf16 gradients, N=8, 5 steps
CONFIG2_FULL_N = 335_000_000
CONFIG2 = FlatConfig(config=2, n=CONFIG2_FULL_N, n_micro=8, steps=5,
                     grad_dtype=torch.bfloat16, grad_std=1e-3)
CONFIG2_SWEEP = [1 << k for k in range(20, 29)] + [CONFIG2_FULL_N]
# config 3: one 4096x4096 linear layer, 4096 tokens per micro-batch, N=4, 3 steps
CONFIG3 = LinearConfig(config=3, tokens=4096, d_in=4096, d_out=4096, n_micro=4, steps=3)


def gpt2xl_block_linears() -> List[Tuple[str, int, int]]:
    """config 4: the four linears of one GPT-2-XL-shaped block as (name, d_in, d_out)."""
    h = 1600
    return [("qkv", h, 3 * h), ("out_proj", h, h), ("fc1", h, 4 * h), ("fc2", 4 * h, h)]


def llama7b_block_linears() -> List[Tuple[str, int, int]]:
    """config 5: the seven linears of one Llama-7B-shaped block as (name, d_in, d_out)."""
    h, f = 4096, 11008
    return [("q", h, h), ("k", h, h), ("v", h, h), ("o", h, h),
            ("gate", h, f), ("up", h, f), ("down", f, h)]


CONFIG4_BLOCKS, CONFIG4_TOKENS, CONFIG4_N_MICRO = 48, 4 * 1024, 8
CONFIG5_BLOCKS, CONFIG5_TOKENS, CONFIG5_N_MICRO, CONFIG5_STEPS = 32, 4096, 16, 2
