"""GPU parity of the drafting kernel over seeded random problems: history lengths on both sides of every
launch-shape threshold (thread count, staging in shared memory, clusters), alphabets from 2 symbols to the
whole vocabulary, copy spans, every flag combination, with and without the precomputed extension table."""
import numpy as np
import pytest

import oracle
import synth
from gpu_util import dev_bf16, dev_i32

pytestmark = pytest.mark.gpu
V = 512


@pytest.fixture(scope="module")
def ctx():
    import paper_2411_03786_b200 as ngs
    W = synth.gaussian_weights(V, 64, 1.0, 1, "W")
    c = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    yield c
    c.close()


@pytest.mark.parametrize("case", range(48))
def test_random_draft_problem(ctx, case):
    import paper_2411_03786_b200 as ngs
    g = np.random.default_rng(9000 + case)
    S = int(g.integers(1, 7))
    Lmax = int([g.integers(1, 64), g.integers(64, 2100), g.integers(2000, 8300), g.integers(8000, 17000),
                g.integers(16000, 70000), g.integers(8100, 8300)][case % 6])
    cap = (Lmax + int(g.integers(0, 200)) + 3) // 4 * 4
    alpha = int(g.choice([2, 3, 6, 40, V]))
    lens = np.array([Lmax if s == 0 else int(g.integers(0, Lmax + 1)) for s in range(S)], np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        h = g.integers(0, alpha, lens[s])
        if g.random() < 0.5 and lens[s] > 40:
            for _ in range(int(lens[s]) // 50):
                a, b, n = int(g.integers(0, lens[s] - 20)), int(g.integers(0, lens[s] - 20)), int(g.integers(4, 20))
                h[b:b + n] = h[a:a + n]
        hist[s, :lens[s]] = h
    n_q = int(g.integers(0, 4))
    qs = [int(q) for q in g.choice([1, 2, 3, 4], n_q, replace=False)]
    B = int(g.integers(1, 33))
    w = int(g.integers(1, 12))
    topk = int(g.integers(1, B + 1))
    k_tab = int(g.integers(1, 17))
    flags = int(g.choice([0, 1, 2, 3, 7, 5])) | (ngs.flag_reserve(int(g.integers(0, B + 1))) if g.random() < 0.3 else 0)
    if case % 4 == 3:
        flags |= ngs.FLAG_PARTIAL_TAIL          # occurrences near the end count too (served by the batch kernels)
        if lens[0] > 30:                        # ... and a periodic tail makes them matter
            per = int(g.integers(1, 7))
            hist[0, lens[0] - 25:lens[0]] = np.resize(hist[0, lens[0] - 25:lens[0] - 25 + per], 25)
    T = np.stack([g.permutation(V)[:k_tab] for _ in range(V)]).astype(np.int32)
    ext = oracle.extend_table(T, w) if g.random() < 0.5 else None
    ctx.set_model_table(dev_i32(T), dev_i32(ext) if ext is not None else None)
    want = oracle.draft_batch(hist, lens, qs, topk, B, w, flags, T)
    got = ctx.draft_context_ngrams(dev_i32(hist), dev_i32(lens), qs, topk, B, w, flags)
    for a, b, name in zip(got, want, ("drafts", "n_drafts", "src", "counts")):
        assert np.array_equal(a.cpu().numpy(), b), name
    assert ctx.get_status() == 0


@pytest.mark.parametrize("alpha,qs,Lmax,flags", [(3, [1], 9000, 3), (40, [2, 1], 12000, 7), (6, [3, 2], 17000, 3),
                                                 (V, [2], 9500, 1), (2, [4, 3], 8400, 5), (6, [1], 16000, 3),
                                                 (40, [1, 2], 10000, 2)])
def test_batch_of_unstaged_histories(ctx, alpha, qs, Lmax, flags):
    """More sequences than SMs, histories of 8K to 17K tokens: the batch kernels (a team of 16 warps per CTA
    up to 16384 tokens, scanner / finisher warps beyond) and the queued grouping of matches, from a few
    matches per warp iteration (queue filled and flushed in mid-scan) to more than a queue holds (grouped
    in place); some cases have more distinct continuations than the table groups in one pass."""
    g = np.random.default_rng(31000 + alpha + Lmax)
    S, B, w, topk, k_tab = 160, 12, 5, 6, 4
    cap = Lmax + 8
    lens = np.array([Lmax if s % 7 == 0 else int(g.integers(Lmax // 2, Lmax + 1)) for s in range(S)], np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        h = g.integers(0, alpha, lens[s])
        for _ in range(int(lens[s]) // 200):
            a, b, n = int(g.integers(0, lens[s] - 20)), int(g.integers(0, lens[s] - 20)), int(g.integers(4, 20))
            h[b:b + n] = h[a:a + n]
        hist[s, :lens[s]] = h
    T = np.stack([g.permutation(V)[:k_tab] for _ in range(V)]).astype(np.int32)
    ctx.set_model_table(dev_i32(T), None)
    want = oracle.draft_batch(hist, lens, qs, topk, B, w, flags, T)
    got = ctx.draft_context_ngrams(dev_i32(hist), dev_i32(lens), qs, topk, B, w, flags)
    for a, b, name in zip(got, want, ("drafts", "n_drafts", "src", "counts")):
        assert np.array_equal(a.cpu().numpy(), b), name
    assert ctx.get_status() == 0


@pytest.mark.parametrize("S,Lmax,alpha,qs,flags", [
    (2400, 2000, 6, [1], 3),         # one warp per sequence, per-warp tables; q = 1 on 6 symbols overflows them (several passes)
    (2400, 300, 40, [3, 2, 1], 3),   # one warp per sequence, a handful of matches each
    (1200, 900, 3, [2, 1], 7),       # two warps per sequence, grouping by the next token only
    (1200, 5000, V, [2], 1),         # ... vocabulary-sized alphabet: hardly any match
    (600, 1500, 6, [4, 3], 5),       # four warps per sequence
    (600, 7000, 6, [1, 2], 3),       # ... about a thousand matches with several hundred distinct continuations: several passes
    (320, 3000, 40, [2, 1], 2),      # eight warps per sequence, no duplicate removal
    (310, 9000, 6, [3, 2], 3),       # eight warps by the batch, unstaged history
    (300, 40000, 6, [2], 3),         # histories too long to stage: scanner and finisher warps, two tables
    (200, 30000, 10, [1, 2], 3),     # ... with more distinct continuations than a table holds: several hand-overs per sequence
    (150, 17000, 40, [3, 1], 7),     # ... fewer sequences than a CTA per SM could take twice
])
def test_batches_across_team_sizes(ctx, S, Lmax, alpha, qs, flags):
    """Batches that fill the GPU more than twice over take the persistent kernels: warp teams (1, 2, 4, 8 or 16 warps,
    by batch size) that stage a history of up to 16384 tokens in shared memory, scanner / finisher warps for longer
    ones; sequences are pulled from a queue, and ragged lengths (down to empty) make the teams take different numbers
    of them.  Two calls in a row: the work queue has to re-arm itself."""
    import paper_2411_03786_b200 as ngs
    g = np.random.default_rng(52000 + S + Lmax)
    B, w, topk, k_tab = 10, 4, 5, 6
    cap = (Lmax + 11) // 4 * 4
    lens = np.array([Lmax if s % 5 == 0 else int(g.integers(0, Lmax + 1)) for s in range(S)], np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        h = g.integers(0, alpha, lens[s])
        for _ in range(int(lens[s]) // 150):
            a, b, n = int(g.integers(0, lens[s] - 20)), int(g.integers(0, lens[s] - 20)), int(g.integers(4, 20))
            h[b:b + n] = h[a:a + n]
        hist[s, :lens[s]] = h
    T = np.stack([g.permutation(V)[:k_tab] for _ in range(V)]).astype(np.int32)
    ext = oracle.extend_table(T, w) if S % 3 == 0 else None
    ctx.set_model_table(dev_i32(T), dev_i32(ext) if ext is not None else None)
    fl = flags | (ngs.flag_reserve(3) if S == 600 else 0)
    want = oracle.draft_batch(hist, lens, qs, topk, B, w, fl, T)
    for rep in range(2):
        got = ctx.draft_context_ngrams(dev_i32(hist), dev_i32(lens), qs, topk, B, w, fl)
        for a, b, name in zip(got, want, ("drafts", "n_drafts", "src", "counts")):
            assert np.array_equal(a.cpu().numpy(), b), name
    assert ctx.get_status() == 0


@pytest.mark.parametrize("S,Lmax,qs,w,flags", [(5, 60, [1, 2], 6, 11), (40, 900, [3, 2, 1], 9, 15), (700, 300, [2], 5, 9),
                                               (3, 12000, [1, 3], 8, 11), (200, 20000, [2, 1], 7, 11), (2, 70000, [4, 2], 16, 9)])
def test_occurrences_with_partial_continuations(ctx, S, Lmax, qs, w, flags):
    """SPEC_FLAG_PARTIAL_TAIL on histories that end in a repeating pattern (period 1 to 2 w): the occurrences that
    decide the draft are the ones closer than w to the end.  Staged teams, scanner / finisher warps, single sequences
    and batches; lengths down to below a window."""
    g = np.random.default_rng(77000 + S + Lmax)
    B, topk, k_tab = 12, 6, 5
    cap = (Lmax + 11) // 4 * 4
    lens = np.array([Lmax if s % 3 == 0 else int(g.integers(0, Lmax + 1)) for s in range(S)], np.int32)
    lens[-1] = min(Lmax, int(g.integers(1, w + 2)))            # shorter than a window
    hist = np.full((S, cap), -1, np.int32)
    n_diff = 0
    for s in range(S):
        h = g.integers(0, 6, lens[s])
        per = int(g.integers(1, 2 * w + 1))
        tail = min(int(lens[s]), per * int(g.integers(2, 6)))
        if tail > per:
            h[lens[s] - tail:] = np.resize(h[lens[s] - tail:lens[s] - tail + per], tail)
        hist[s, :lens[s]] = h
    T = np.stack([g.permutation(V)[:k_tab] for _ in range(V)]).astype(np.int32)
    ctx.set_model_table(dev_i32(T), None)
    want = oracle.draft_batch(hist, lens, qs, topk, B, w, flags, T)
    plain = oracle.draft_batch(hist, lens, qs, topk, B, w, flags & ~8, T)
    assert not np.array_equal(want[0], plain[0])                 # the flag changes the drafts on these histories
    got = ctx.draft_context_ngrams(dev_i32(hist), dev_i32(lens), qs, topk, B, w, flags)
    for a, b, name in zip(got, want, ("drafts", "n_drafts", "src", "counts")):
        assert np.array_equal(a.cpu().numpy(), b), name
    assert ctx.get_status() == 0
