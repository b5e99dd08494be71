"""Host-side helpers for running one process per GPU.

The speculation step shards by sequences: every rank owns a contiguous block of sequences and a
replica of the head, and no data crosses ranks on the hot path.  The only collectives are the
barrier around the timed region and the reduction of timings (max over ranks) and token counts
(sum over ranks).  Works with any torch.distributed backend (NCCL on GPUs, gloo on CPU).
"""
from __future__ import annotations

import torch


def shard_sequences(n_sequences: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous block ``(first, count)`` of sequences owned by ``rank``; blocks differ by at most one."""
    base, extra = divmod(n_sequences, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def reduce_max_sum(maxima, sums, device="cpu"):
    """All-reduce ``maxima`` with MAX and ``sums`` with SUM across ranks; returns two lists of floats.

    Without an initialised process group (single process) the inputs come back unchanged.
    """
    import torch.distributed as dist
    maxima, sums = [float(x) for x in maxima], [float(x) for x in sums]
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return maxima, sums
    m = torch.tensor(maxima, dtype=torch.float64, device=device)
    s = torch.tensor(sums, dtype=torch.float64, device=device)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return m.tolist(), s.tolist()


def whole_job_throughput(tokens_this_rank: float, ms_this_rank: float, device="cpu") -> tuple[float, float]:
    """``(tokens per second of the whole job, slowest rank's ms)``: all ranks' tokens over the slowest rank's time."""
    (ms,), (tokens,) = reduce_max_sum([ms_this_rank], [tokens_this_rank], device)
    return tokens / (ms / 1e3), ms
