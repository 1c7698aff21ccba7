"""Host-side logic for running the attention path on several GPUs of one node.

Every (batch row, head) is an independent unit of the step-k attention and the tile plan is the same
for all of them, so the path shards without any collective on the data path: each rank owns its batch
rows, builds the same plan, and launches the same kernels on its own GPU.  What ranks exchange is only
the measured time (maximum over ranks) for reporting.
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def split_units(n_units: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous range [begin, end) of the n_units (batch row, head) units owned by `rank`:
    sizes differ by at most one, every unit belongs to exactly one rank."""
    if not (0 <= rank < world) or n_units < 0:
        raise ValueError("bad rank/world/n_units")
    base, extra = divmod(n_units, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def rank_seed(seed: int, rank: int) -> int:
    """Distinct input streams per rank (weak scaling: every rank has its own batch)."""
    return int(seed) + 7_919 * int(rank)


def max_over_ranks(values: List[float], device=None) -> List[float]:
    """Element-wise maximum of per-rank measurements over the default process group
    (identity when torch.distributed is not initialised)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_rate(work_per_rank: float, world: int, slowest_ms: float) -> float:
    """Aggregate rate of a weak-scaling run: every rank did `work_per_rank`, the job took as long as
    its slowest rank."""
    return world * work_per_rank / (slowest_ms * 1e-3)
