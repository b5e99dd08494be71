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


def sharded_verify(ctx, hidden, vocab_offset: int, V_total: int, with_max: bool = False):
    """Verification when every rank holds a slice of the vocabulary (``ctx`` was created with this
    rank's rows of the unembedding, which start at token id ``vocab_offset``).

    Each rank computes per-row (logit, id) keys over its slice; one all-reduce with MAX over the
    int64 keys picks the winner across ranks (lowest global id on exact ties); the keys are then
    unpacked.  Without a process group this is a single-shard verify.
    """
    import torch.distributed as dist
    from .binding import unpack_keys
    keys = ctx.verify_lmhead_keys(hidden, vocab_offset)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(keys, op=dist.ReduceOp.MAX)
    return unpack_keys(keys, V_total, with_max)


def all_gather_rows(local: torch.Tensor, n_total: int, rank: int, world: int) -> torch.Tensor:
    """Stitches per-rank row slices (rank r owns ``shard_sequences(n_total, r, world)``) into the whole
    ``[n_total, ...]`` array on every rank: one all-gather of equally padded slices, into local buffers."""
    import torch.distributed as dist
    first, count = shard_sequences(n_total, rank, world)
    assert local.shape[0] == count, "this rank's slice has the wrong number of rows"
    if not (dist.is_available() and dist.is_initialized()) or world == 1:
        return local.clone()
    most = (n_total + world - 1) // world
    padded = torch.zeros((most,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    padded[:count] = local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    return torch.cat([parts[r][:shard_sequences(n_total, r, world)[1]] for r in range(world)], dim=0)


def sharded_table_build(ctx, k_tab: int, w_ext: int, rank: int, world: int, rows: torch.Tensor | None = None):
    """Model bigram table with the rows split over the ranks (every rank holds the whole head):
    each rank contracts its ``V / world`` rows, one all-gather of the ``[rows, k_tab]`` int32 slices
    gives every rank the complete table, and the extension is then derived locally.
    Returns ``(table[V, k_tab], ext[V, k_tab, w_ext] or None)``; the context adopts them when w_ext > 0."""
    V = ctx.V
    first, count = shard_sequences(V, rank, world)
    tab = torch.zeros((V, k_tab), dtype=torch.int32, device=ctx._keep[0].device)
    ctx.build_model_ngram_table_rows(k_tab, first, count, tab, rows=rows)
    whole = all_gather_rows(tab[first:first + count].contiguous(), V, rank, world)
    if w_ext > 0:
        return whole, ctx.extend_model_table(whole, w_ext)
    ctx.set_model_table(whole)
    return whole, None


def pack_key(value: float, token_id: int) -> int:
    """Host-side statement of the shard key format (for tests and debugging): a signed 64-bit integer
    that is larger for a larger fp32 logit and, for equal logits, for a smaller token id."""
    import struct
    (u,) = struct.unpack("<I", struct.pack("<f", value))
    u = (~u & 0xFFFFFFFF) if u & 0x80000000 else (u | 0x80000000)
    k = ((u << 32) | (~token_id & 0xFFFFFFFF)) ^ 0x8000000000000000
    return k - (1 << 64) if k >= (1 << 63) else k


def unpack_key(key: int) -> tuple[float, int]:
    import struct
    k = (key + (1 << 64)) % (1 << 64) ^ 0x8000000000000000
    u = k >> 32
    u = (u & 0x7FFFFFFF) if u & 0x80000000 else (~u & 0xFFFFFFFF)
    return struct.unpack("<f", struct.pack("<I", u))[0], (~k) & 0xFFFFFFFF
