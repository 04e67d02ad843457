"""Data-parallel sharding of decode batches across ranks (one process per GPU).

Sequences are independent units, so the path shards by sequence with no
data-path collective: every rank draws and serves its own batch. The only
communication is the benchmark's bookkeeping: the step time is the max over
ranks and the work is the sum over ranks.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of rank ``rank``'s batch (rank 0 keeps the single-GPU seed)."""
    return base_seed + 1000 * rank


def shard_sequences(n_sequences: int, rank: int, world: int) -> range:
    """Contiguous slice of a global batch owned by ``rank`` (sizes differ by at most 1)."""
    base, extra = divmod(n_sequences, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def aggregate(times_ms, work, device="cpu"):
    """``times_ms``: per-rank timings -> elementwise max over ranks;
    ``work``: per-rank work counters -> elementwise sum over ranks."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    w = torch.tensor(list(work), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [float(x) for x in w.tolist()]
