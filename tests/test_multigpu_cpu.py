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


def test_shard_keys_order_by_logit_then_lower_token_id():
    vals = [-3.5, -0.0, 0.0, 1e-30, 2.25, 2.25, 1e30]
    ids = [7, 3, 9, 1, 500, 20, 0]
    keys = [multigpu.pack_key(v, i) for v, i in zip(vals, ids)]
    for (v, i), k in zip(zip(vals, ids), keys):
        v2, i2 = multigpu.unpack_key(k)
        assert v2 == np.float32(v) and i2 == i and -(1 << 63) <= k < (1 << 63)
    best = max(range(len(keys)), key=lambda j: keys[j])
    assert best == 6
    assert multigpu.pack_key(2.25, 20) > multigpu.pack_key(2.25, 500)        # equal logits: the lower id wins
    assert multigpu.pack_key(-1.0, 5) < multigpu.pack_key(-0.5, 5) < multigpu.pack_key(0.5, 5)


def _reduce_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "owns" token ids [100 r, 100 r + 100): its best (logit, id) per row, as shard keys
    g = np.random.default_rng(rank)
    vals = g.standard_normal(16).astype(np.float32)
    vals[3] = 1.5                                    # an exact tie across ranks: rank 0's id is lower
    ids = 100 * rank + g.integers(0, 100, 16)
    keys = torch.tensor([multigpu.pack_key(float(v), int(i)) for v, i in zip(vals, ids)], dtype=torch.int64)
    dist.all_reduce(keys, op=dist.ReduceOp.MAX)
    out.put((rank, vals.tolist(), ids.tolist(), keys.tolist()))
    dist.destroy_process_group()


def test_max_all_reduce_of_shard_keys_picks_the_global_argmax():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_reduce_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, v0, i0, k0), (_, v1, i1, k1) = res
    assert k0 == k1
    for j in range(16):
        v, i = multigpu.unpack_key(k0[j])
        want = (v0[j], i0[j]) if (v0[j] > v1[j] or (v0[j] == v1[j] and i0[j] < i1[j])) else (v1[j], i1[j])
        assert (v, i) == (np.float32(want[0]), want[1])


def _table_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    import synth
    V, d, k = 37, 16, 3                                   # odd V: the two slices differ in size
    E = synth.gaussian_weights(V, d, 1.0, 3, "E")
    W = synth.gaussian_weights(V, d, 1.0, 3, "W")
    first, count = multigpu.shard_sequences(V, rank, world)
    mine, _ = oracle.model_table(E, W, k, rows=np.arange(first, first + count))     # this rank's rows only
    whole = multigpu.all_gather_rows(torch.from_numpy(mine), V, rank, world)
    out.put((rank, whole.numpy().tolist()))
    dist.destroy_process_group()


def test_two_gloo_ranks_stitch_their_table_slices_into_the_whole_table():
    import oracle
    import synth
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_table_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    E = synth.gaussian_weights(37, 16, 1.0, 3, "E")
    W = synth.gaussian_weights(37, 16, 1.0, 3, "W")
    whole, _ = oracle.model_table(E, W, 3)
    assert res[0][1] == res[1][1] == whole.tolist()
    # single process: the slice is the table
    one = multigpu.all_gather_rows(torch.from_numpy(whole), 37, 0, 1)
    assert one.numpy().tolist() == whole.tolist()


def test_bench_refuses_to_run_fewer_ranks_than_asked():
    """`bench.py --gpus N` without a launcher starts N ranks itself - and fails loudly when the machine does not
    show N GPUs (here: none), instead of quietly running one rank."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "1"], capture_output=True, text=True,
                       env=env, timeout=300)
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        return                                             # a machine with two GPUs would simply run it
    assert r.returncode != 0
    assert "refusing to run fewer ranks than asked" in (r.stderr + r.stdout)
