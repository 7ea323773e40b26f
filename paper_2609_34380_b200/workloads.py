"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors and index lists; it holds none of the
method's arithmetic (no split, no reconstruction, no product), so that both the
CUDA path and the CPU oracle can be fed from it without sharing logic.

The paper serves MoE and dense LLMs whose projection weights have a small range
and switches mode in long, bursty windows (sections "Mapper: Semi-Unified Memory
Abstraction" and the evaluation's switching-overhead table).  Real checkpoints and
traces are not available offline, so weights are FP16 roundings of
0.02 * N(0,1), activations FP16 roundings of N(0,1), and the mode schedule is a
seeded alternation of Poisson-length stretches.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

# (N, K) = (out_features, in_features) per linear, as in torch.nn.Linear.weight
TINY: Dict[str, Tuple[int, int]] = {"linear": (512, 512)}
LLAMA7B: Dict[str, Tuple[int, int]] = {
    "qkv": (12288, 4096),
    "o": (4096, 4096),
    "gate_up": (22016, 4096),
    "down": (4096, 11008),
}
MIXTRAL_EXPERT: Dict[str, Tuple[int, int]] = {"gate_up": (28672, 4096), "down": (4096, 14336)}
MIXTRAL_EXPERTS = 8
MIXTRAL_TOKENS = 256
DECODER70: Dict[str, Tuple[int, int]] = {
    "qkv": (10240, 8192),
    "o": (8192, 8192),
    "gate_up": (57344, 8192),
    "down": (8192, 28672),
}
DECODER70_LAYERS = 32

DECODE_M = (1, 8, 32)
PREFILL_M = (512, 2048, 8192)
STEP_M = (1, 16, 64, 256)


def _generator(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def weights(n: int, k: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    """FP16 [n][k] = round_fp16(std * N(0,1)).  The stream depends on the device kind,
    so a test draws once and copies the tensor to wherever else it is needed."""
    g = _generator(seed, device)
    w = torch.randn((n, k), generator=g, device=device, dtype=torch.float32)
    return (w * std).to(torch.float16)


def activations(m: int, k: int, seed: int, device="cpu") -> torch.Tensor:
    """FP16 [m][k] = round_fp16(N(0,1))."""
    g = _generator(seed, device)
    return torch.randn((m, k), generator=g, device=device, dtype=torch.float32).to(torch.float16)


def top2_routing(tokens: int, experts: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Each token goes to two distinct experts drawn uniformly (partial Fisher-Yates).

    Returns (token_of_row, expert_of_row), int32 arrays of length 2*tokens with
    token_of_row[a] = a // 2.
    """
    rng = np.random.default_rng(seed)
    expert_of_row = np.empty(2 * tokens, np.int32)
    for t in range(tokens):
        perm = np.arange(experts)
        for j in range(2):
            pick = j + int(rng.integers(0, experts - j))
            perm[j], perm[pick] = perm[pick], perm[j]
        expert_of_row[2 * t] = perm[0]
        expert_of_row[2 * t + 1] = perm[1]
    token_of_row = (np.arange(2 * tokens) // 2).astype(np.int32)
    return token_of_row, expert_of_row


def mode_schedule(steps: int = 256, seed: int = 5555, full_mean: float = 12.0,
                  fast_mean: float = 20.0) -> List[int]:
    """Bursty per-step mode list (1 = full, 0 = fast), starting in full mode.

    Stretch lengths are 1 + Poisson(mean): long fast bursts between full-mode
    stretches, about 62 % of steps fast -- between the 47 % and 79 % the paper's
    switching-overhead table reports for its two switching models.
    """
    rng = np.random.default_rng(seed)
    out: List[int] = []
    mode = 1
    while len(out) < steps:
        n = 1 + int(rng.poisson(full_mean if mode == 1 else fast_mean))
        out.extend([mode] * n)
        mode ^= 1
    return out[:steps]


def sample_entries(m: int, n: int, count: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Seeded random (row, column) output positions for sampled checks."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, m, count).astype(np.int64), rng.integers(0, n, count).astype(np.int64)


def as_words(t: torch.Tensor) -> np.ndarray:
    """FP16 tensor -> host uint16 words (a view of the bits, no conversion)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def with_outlier(w: torch.Tensor, value: float = 3.0) -> torch.Tensor:
    """Copy of w with one large element, which pushes a tensor out of E4M3 range."""
    w = w.clone()
    w.view(-1)[0] = value
    return w
