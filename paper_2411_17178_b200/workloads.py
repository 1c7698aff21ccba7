"""Seeded synthetic inputs and the five benchmark workloads.

This module is the only code shared by the CPU oracle's tests and the CUDA path's
tests/bench.  It holds shapes, seeds and random-number generation only: no mask, no
softmax, no attention arithmetic.  Tensors are generated on the host so both sides
see identical bits.

Shapes follow the VAR coarse-to-fine schedule of the paper's Section 2: scale k has
s_k^2 tokens and the step-k attention map is [s_k^2, sum_{i<=k} s_i^2].  The paper's
measurements use VAR activations on ImageNet; neither is available offline, so
N(0,1) bf16 tensors of the same shapes stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

HEAD_DIM = 64

SCALES_256 = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)            # paper, "MDWA implementation details"
SCALES_512 = (1, 2, 3, 4, 6, 9, 13, 18, 24, 32)
SCALES_2K = (1, 2, 3, 4, 6, 9, 13, 18, 24, 32, 48, 64, 96, 128)


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (index = 1-based position in the config list)."""
    index: int
    name: str
    scales: Tuple[int, ...]
    steps: Tuple[int, ...]            # 1-based step indices run per layer
    n_layers: int
    n_heads: int
    batch_pairs: int                  # B: the batch is 2B rows, first B conditional
    share_cfg: bool                   # CFG output sharing at every step
    rho: Tuple[int, int] = (1, 4)     # relative window radius (numerator, denominator)
    key_head_scale: bool = False      # config 4: K multiplied per head by U[0.5, 2]
    rho_sweep: Tuple[Tuple[int, int], ...] = field(default_factory=tuple)


WORKLOADS = {
    1: Workload(1, "var-d16-256px-step10", SCALES_256, (10,), 1, 16, 1, False),
    2: Workload(2, "var-d16-256px-schedule", SCALES_256, tuple(range(1, 11)), 16, 16, 8, True),
    3: Workload(3, "var-d30-256px-schedule", SCALES_256, tuple(range(1, 11)), 30, 30, 32, True),
    4: Workload(4, "var-d36-512px-schedule", SCALES_512, tuple(range(1, 11)), 36, 36, 8, True,
                key_head_scale=True),
    5: Workload(5, "2k-stress-step14", SCALES_2K, (14,), 1, 16, 1, False,
                rho_sweep=((1, 8), (1, 4), (1, 2))),
}


def tokens_per_scale(scales: Sequence[int]) -> List[int]:
    return [int(s) * int(s) for s in scales]


def cache_len(scales: Sequence[int], step_k: int) -> int:
    """Rows of the cumulative K/V cache visible at 1-based step k."""
    return sum(tokens_per_scale(scales)[:step_k])


def seed_for(config: int, layer: int, step: int, tensor: int) -> int:
    """tensor: 0 = Q (per step), 1 = K, 2 = V (step 0: one cumulative cache per layer)."""
    return 1_000_000 * config + 1_000 * layer + 10 * step + tensor


def randn_bf16(shape: Sequence[int], seed: int) -> torch.Tensor:
    """N(0,1) drawn in fp32 on the host with a fixed seed, rounded to bf16 (RNE)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return torch.randn(*shape, generator=g, dtype=torch.float32).to(torch.bfloat16)


def head_scales(n_heads: int, seed: int = 4_999_999) -> torch.Tensor:
    """Per-head multipliers U[0.5, 2] used by config 4 to vary softmax sharpness."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return 0.5 + 1.5 * torch.rand(n_heads, generator=g, dtype=torch.float32)


def make_q(wl: Workload, layer: int, step_k: int, batch_rows: Optional[int] = None) -> torch.Tensor:
    """Q of step k: [2B, H, n_k, 64] bf16 (host)."""
    rows = 2 * wl.batch_pairs if batch_rows is None else batch_rows
    n_k = wl.scales[step_k - 1] ** 2
    return randn_bf16((rows, wl.n_heads, n_k, HEAD_DIM), seed_for(wl.index, layer, step_k, 0))


def make_kv(wl: Workload, layer: int, batch_rows: Optional[int] = None,
            max_step: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Cumulative K and V caches of one layer: [2B, H, L, 64] bf16 (host); step k reads rows [0, L_k)."""
    rows = 2 * wl.batch_pairs if batch_rows is None else batch_rows
    last = max(wl.steps) if max_step is None else max_step
    L = cache_len(wl.scales, last)
    shape = (rows, wl.n_heads, L, HEAD_DIM)
    if wl.key_head_scale:
        g = torch.Generator(device="cpu")
        g.manual_seed(seed_for(wl.index, layer, 0, 1))
        k32 = torch.randn(*shape, generator=g, dtype=torch.float32)
        k = (k32 * head_scales(wl.n_heads).view(1, -1, 1, 1)).to(torch.bfloat16)
    else:
        k = randn_bf16(shape, seed_for(wl.index, layer, 0, 1))
    v = randn_bf16(shape, seed_for(wl.index, layer, 0, 2))
    return k, v


def small_workload(scales: Sequence[int], n_heads: int = 2, batch_pairs: int = 1,
                   share_cfg: bool = False, index: int = 90, rho=(1, 4)) -> Workload:
    """Ad-hoc workload for tests on tiny scale lists."""
    K = len(scales)
    return Workload(index, "test-" + "-".join(map(str, scales)), tuple(scales),
                    tuple(range(1, K + 1)), 1, n_heads, batch_pairs, share_cfg, rho=tuple(rho))
