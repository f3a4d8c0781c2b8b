"""Row sharding for several GPUs: rows are independent, so ranks take contiguous row blocks and the
data path has no collective. Pure host logic (no CUDA, no arithmetic of the path)."""
from __future__ import annotations

from typing import Tuple


def shard_rows(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Half-open row range [lo, hi) of `rank` when B rows are split as evenly as possible over `world` ranks."""
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(seconds: float, dist, device=None) -> float:
    """Slowest rank's time: the figure a multi-GPU throughput is computed from."""
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])
