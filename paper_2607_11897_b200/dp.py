"""Data-parallel plumbing for N > 1 processes (one per GPU).

The path shards over (batch, head) pairs with no data-path collective: every pair is an
independent recurrence.  A rank owns a contiguous block of batch elements; the only
communication is the barrier and the max-over-ranks reduction of the measured time.
"""
import torch
import torch.distributed as dist


def rank_batch_range(batch_per_rank: int, rank: int):
    """Global batch indices owned by `rank` when every rank carries `batch_per_rank` elements (weak scaling)."""
    return range(rank * batch_per_rank, (rank + 1) * batch_per_rank)


def split_batch(total_batch: int, world: int, rank: int):
    """Contiguous block of a fixed global batch owned by `rank` (strong scaling); blocks differ by at most one."""
    base, extra = divmod(total_batch, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a per-rank scalar over the process group (identity without one)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: int, world: int, seconds_max: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / seconds_max
