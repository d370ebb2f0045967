"""Row sharding for multi-GPU runs: rows (frames) are independent under per-row activation
scales, so a batch is split across ranks with replicated weights and no data-path collective."""
from __future__ import annotations

from typing import Tuple


def row_shard(M: int, rank: int, world: int, align: int = 128) -> Tuple[int, int]:
    """[begin, end) of rank's rows: contiguous, sizes differ by at most one `align`-row tile."""
    tiles = (M + align - 1) // align
    base, extra = divmod(tiles, world)
    t0 = rank * base + min(rank, extra)
    t1 = t0 + base + (1 if rank < extra else 0)
    return min(t0 * align, M), min(t1 * align, M)


def aggregate_throughput(units_per_rank, max_seconds: float) -> float:
    """Whole-job throughput: all ranks' units over the slowest rank's time."""
    return sum(units_per_rank) / max_seconds
