"""The N > 1 host logic on CPU: two gloo ranks shard sequences, run the oracle's step on their
shard, and reduce timings (max) and tokens (sum) the way bench.py does."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2411_03786_b200 import multigpu


def test_shards_partition_the_sequences():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            blocks = [multigpu.shard_sequences(n, r, world) for r in range(world)]
            assert sum(c for _, c in blocks) == n
            assert all(blocks[i][0] + blocks[i][1] == blocks[i + 1][0] for i in range(world - 1))
            assert max(c for _, c in blocks) - min(c for _, c in blocks) <= 1


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    import synth
    S, L, V, B, w = 6, 200, 50, 4, 3
    hist, lens, _ = synth.zipf_histories(S, L, V, 1.1, 0.3, seed=5, cap=L + 8)
    first, count = multigpu.shard_sequences(S, rank, world)
    h, l = hist[first:first + count].copy(), lens[first:first + count].copy()
    drafts, nd, _, _ = oracle.draft_batch(h, l, [1], B, B, w, 1, None)
    P = np.concatenate([drafts.clip(min=0), np.zeros((count, B, 1), np.int32)], axis=2)   # accept everything drafted
    acc, _, _ = oracle.accept_commit(drafts, nd, P, h, l)
    tokens = float((acc + 1).sum())
    value, ms = multigpu.whole_job_throughput(tokens, 10.0 * (rank + 1))
    dist.barrier()
    out.put((rank, tokens, value, ms))
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_like_the_benchmark():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    total = res[0][1] + res[1][1]
    assert total > 0
    for _, _, value, ms in res:
        assert ms == 20.0                                  # slowest rank
        assert abs(value - total / 0.020) < 1e-6           # whole-job tokens over the slowest rank's time
