"""Host-side plumbing for running the pass on several GPUs of one node.

Three ways the pass shards, one process per GPU:

* by stream - dialogue streams are independent: every rank owns a set of streams on its own
  GPU and there is no collective on the data path (``owned_streams``, ``split_streams``);
* by K/V plane - under a tensor- or pipeline-parallel model every rank holds some layers or
  some KV heads of every stream.  The scores ``E`` are per token, not per plane, so every
  rank keeps a replica of them, runs the same selection and gets the same keep list; it then
  compacts the planes it owns.  No collective either (``plane_shard``);
* by vocabulary - under a vocabulary-parallel LM head every rank holds a column range of the
  logits.  It reduces its range to one (max, sum exp) pair and a target logit per row
  (``sirllm_score_partial``); the ranks exchange those few bytes per row
  (``exchange_vocab_partials``: one all-gather, one all-reduce) and finish the scores with
  ``sirllm_score_pairs`` (``vocab_ranges``).

What else crosses ranks is bookkeeping: the reduction of per-rank timings / counts for a
report.  This module holds no arithmetic of the method.
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


def vocab_ranges(vocab: int, world: int) -> list:
    """Contiguous, balanced column ranges ``[(v0, v1), ...]``, one per rank, covering the
    vocabulary (the layout of a vocabulary-parallel LM head)."""
    base, extra = divmod(vocab, world)
    out, v0 = [], 0
    for r in range(world):
        v1 = v0 + base + (1 if r < extra else 0)
        out.append((v0, v1))
        v0 = v1
    return out


def plane_shard(n_layers: int, n_kv_heads: int, world: int, rank: int, by: str = "layers"):
    """The planes one rank owns when the K/V cache is split across ranks: ``(layers, heads)``
    as two ranges, splitting either the layers (pipeline-style) or the KV heads (tensor-style)
    evenly.  The rank's configuration is the full one with ``n_layers`` / ``n_kv_heads``
    replaced by the lengths of these ranges."""
    if by == "layers":
        return split_streams(n_layers, world, rank), range(n_kv_heads)
    if by == "heads":
        return range(n_layers), split_streams(n_kv_heads, world, rank)
    raise ValueError("by must be 'layers' or 'heads'")


def exchange_vocab_partials(pairs_local: torch.Tensor, target_local: torch.Tensor, group=None):
    """Combines the ranks' shares of vocabulary-parallel scoring.

    ``pairs_local`` is this rank's ``[rows, 2]`` (max, sum exp) pairs, ``target_local`` its
    ``[rows]`` target logits (0 where the token's column belongs to another rank).  Returns
    ``pairs [rows, world, 2]`` (all-gather) and ``target [rows]`` (sum over ranks: exactly one
    rank contributes a non-zero value per row), ready for ``sirllm_score_pairs``.  Message
    size: 12 bytes per row and rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return pairs_local.unsqueeze(1).contiguous(), target_local.clone()
    world = dist.get_world_size(group)
    gathered = [torch.empty_like(pairs_local) for _ in range(world)]
    dist.all_gather(gathered, pairs_local.contiguous(), group=group)
    target = target_local.clone()
    dist.all_reduce(target, op=dist.ReduceOp.SUM, group=group)
    return torch.stack(gathered, dim=1).contiguous(), target
