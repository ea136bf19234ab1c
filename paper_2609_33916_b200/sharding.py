"""How a workload is split across GPUs: (batch, head) pairs are independent, so each
rank takes a contiguous block of heads and no collective is needed on the data path."""
from __future__ import annotations


def head_shard(total_heads: int, world: int, rank: int) -> tuple[int, int]:
    """(first head, number of heads) of `rank`: contiguous blocks, sizes differing by at
    most one, the larger blocks on the lower ranks."""
    if world <= 0 or not (0 <= rank < world) or total_heads < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total_heads, world)
    count = base + (1 if rank < extra else 0)
    start = rank * base + min(rank, extra)
    return start, count


def aggregate_rate(units_per_rank: list[float], seconds_per_rank: list[float]) -> float:
    """Whole-job rate: all ranks' units over the slowest rank's time."""
    return sum(units_per_rank) / max(seconds_per_rank)
