"""Host-side plumbing for running the pass on several GPUs of one node.

Dialogue streams are independent, so the pass shards by stream: every rank owns a set of
streams on its own GPU and there is no collective on the data path.  What crosses ranks is
bookkeeping only: which global stream ids a rank owns (so that seeded inputs differ between
ranks) and the reduction of per-rank timings / counts for a report.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def owned_streams(streams_per_rank: int, rank: int) -> range:
    """Global ids of the streams a rank hosts when every rank hosts ``streams_per_rank``
    (weak scaling: the job has ``world * streams_per_rank`` streams)."""
    return range(rank * streams_per_rank, (rank + 1) * streams_per_rank)


def split_streams(total_streams: int, world: int, rank: int) -> range:
    """Contiguous, balanced share of ``total_streams`` for ``rank`` (strong scaling)."""
    base, extra = divmod(total_streams, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def _reduce(value: float, op, device) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t[0])


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: multi-GPU numbers are the max over ranks."""
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)
