"""GPU parity of the incremental context index: over hundreds of decode steps the indexed drafting must give,
bit for bit, what the scan gives and what the oracle gives, while the index is only ever updated with the
windows that each step's committed tokens completed."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import dev_bf16, dev_i32

pytestmark = pytest.mark.gpu
V = 512


@pytest.fixture(scope="module")
def ngs():
    import paper_2411_03786_b200 as m
    return m


@pytest.fixture(scope="module")
def ctx(ngs):
    W = synth.gaussian_weights(V, 64, 1.0, 1, "W")
    c = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    yield c
    c.close()


def predictions(g, drafts, nd, w, alpha):
    """Model predictions that accept a random prefix of a random draft row (0 .. w tokens) and then a random token."""
    S, B, _ = drafts.shape
    P = g.integers(0, alpha, (S, B, w + 1)).astype(np.int32)
    for s in range(S):
        if nd[s] > 0:
            b, a = int(g.integers(0, nd[s])), int(g.integers(0, w + 1))
            P[s, b, :a] = drafts[s, b, :a]
    return P


def decode(ngs, ctx, hist0, lens0, qs, topk, B, w, flags, steps, alpha, seed, T):
    g = np.random.default_rng(seed)
    hist_h, lens_h = hist0.copy(), lens0.copy()
    hist, lens = dev_i32(hist_h), dev_i32(lens_h)
    ext = oracle.extend_table(T, w)
    ctx.set_model_table(dev_i32(T), dev_i32(ext))
    index = ctx.context_index_build(hist, lens, qs, w, flags & ngs.FLAG_KEY_NEXT_TOKEN)
    for step in range(steps):
        want = oracle.draft_batch(hist_h, lens_h, qs, topk, B, w, flags, T)
        got_i = ctx.draft_context_ngrams_indexed(index, hist, lens, qs, topk, B, w, flags)
        got_s = ctx.draft_context_ngrams(hist, lens, qs, topk, B, w, flags)
        for a, b, c, name in zip(got_i, got_s, want, ("drafts", "n_drafts", "src", "counts")):
            assert np.array_equal(a.cpu().numpy(), c), f"step {step}: indexed {name} differs from the oracle"
            assert np.array_equal(b.cpu().numpy(), c), f"step {step}: scanned {name} differs from the oracle"
        P = predictions(g, want[0], want[1], w, alpha)
        acc_r, best_r, com_r = oracle.accept_commit(want[0], want[1], P, hist_h, lens_h)
        acc, best, com = ctx.accept_and_commit_indexed(index, got_i[0], got_i[1], dev_i32(P), hist, lens)
        assert np.array_equal(acc.cpu().numpy(), acc_r) and np.array_equal(com.cpu().numpy(), com_r)
        assert np.array_equal(lens.cpu().numpy(), lens_h)
    assert np.array_equal(hist.cpu().numpy(), hist_h)
    return index, hist, lens, hist_h, lens_h


@pytest.mark.parametrize("name,steps", [("C1", 220), ("C3", 200), ("C5", 200)])
def test_indexed_drafting_equals_scan_and_oracle_over_a_decode(ngs, ctx, name, steps):
    c = synth.config(name)
    S = min(c["S"], 8)
    w = c["w"]
    hist, lens, _ = synth.zipf_histories(S, c["L"], c["V"], c["zipf"], c["copy"], c["seed"], cap=c["L"] + steps * (w + 1) + 8)
    hist = np.where(hist >= 0, hist % V, -1).astype(np.int32)       # token ids folded into the small context's vocabulary
    g = np.random.default_rng(c["seed"])
    T = np.stack([g.permutation(V)[:c["k_tab"]] for _ in range(V)]).astype(np.int32)
    decode(ngs, ctx, hist, lens, list(c["qs"]), c["topk"], c["B"], w, 3, steps, V, c["seed"] + 7, T)
    assert ctx.get_status() == 0


@pytest.mark.parametrize("flags", [3, 7, 1 | (2 << 8), 2])
def test_indexed_drafting_on_small_alphabets_and_ragged_lengths(ngs, ctx, flags):
    """Heavy repetition (3 symbols), sequences that start empty or shorter than a window, every flag combination
    (duplicates kept or dropped, next-token keys, reserved rows)."""
    g = np.random.default_rng(flags)
    S, cap, w, B = 6, 700, 4, 12
    lens = np.array([0, 1, 3, 40, 150, 300], np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, 3, lens[s])
    T = np.stack([g.permutation(V)[:5] for _ in range(V)]).astype(np.int32)
    decode(ngs, ctx, hist, lens, [2, 1, 3], 5, B, w, flags, 60, 3, 100 + flags, T)
    assert ctx.get_status() == 0


def test_index_out_of_step_or_too_crowded_falls_back_to_the_scan(ngs, ctx):
    g = np.random.default_rng(11)
    S, cap, w, B, qs, topk = 3, 12000, 4, 16, [1, 2], 6
    lens = np.array([9000, 5000, 200], np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, V, lens[s])
    hist[0, :9000:2] = 7                       # every other token is the query token: thousands of groups for q = 1
    hist[0, 8999] = 7
    T = np.stack([g.permutation(V)[:4] for _ in range(V)]).astype(np.int32)
    index, d_hist, d_lens, hist_h, lens_h = decode(ngs, ctx, hist, lens, qs, topk, B, w, 3, 5, V, 12, T)
    # a commit by the plain call moves the histories without the index: the indexed call must notice and scan
    want = oracle.draft_batch(hist_h, lens_h, qs, topk, B, w, 3, T)
    P = predictions(g, want[0], want[1], w, V)
    oracle.accept_commit(want[0], want[1], P, hist_h, lens_h)
    ctx.accept_and_commit(dev_i32(want[0]), dev_i32(want[1]), dev_i32(P), d_hist, d_lens)
    for rep in range(3):
        want = oracle.draft_batch(hist_h, lens_h, qs, topk, B, w, 3, T)
        got = ctx.draft_context_ngrams_indexed(index, d_hist, d_lens, qs, topk, B, w, 3)
        for a, c, name in zip(got, want, ("drafts", "n_drafts", "src", "counts")):
            assert np.array_equal(a.cpu().numpy(), c), name
        P = predictions(g, want[0], want[1], w, V)
        oracle.accept_commit(want[0], want[1], P, hist_h, lens_h)
        ctx.accept_and_commit_indexed(index, got[0], got[1], dev_i32(P), d_hist, d_lens)   # stays out of step: no update, no harm
    assert np.array_equal(d_hist.cpu().numpy(), hist_h)
    # rebuilding brings the index back
    index = ctx.context_index_build(d_hist, d_lens, qs, w)
    want = oracle.draft_batch(hist_h, lens_h, qs, topk, B, w, 3, T)
    got = ctx.draft_context_ngrams_indexed(index, d_hist, d_lens, qs, topk, B, w, 3)
    for a, c in zip(got, want):
        assert np.array_equal(a.cpu().numpy(), c)
    assert ctx.get_status() == 0
    # argument checks: another buffer, another width, a query length that was not indexed
    with pytest.raises(ngs.SpecError, match="registered"):
        ctx.draft_context_ngrams_indexed(torch.empty_like(index), d_hist, d_lens, qs, topk, B, w, 3)
    with pytest.raises(ngs.SpecError, match="built with"):
        ctx.draft_context_ngrams_indexed(index, d_hist, d_lens, qs, topk, B, w + 1, 3)
    with pytest.raises(ngs.SpecError, match="not built for q = 3"):
        ctx.draft_context_ngrams_indexed(index, d_hist, d_lens, [3], topk, B, w, 3)


def test_commit_that_does_not_fit_leaves_history_and_index_untouched(ngs, ctx):
    S, cap, w, B = 2, 64, 4, 4
    hist = np.full((S, cap), -1, np.int32)
    lens = np.array([62, 30], np.int32)
    g = np.random.default_rng(5)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, 4, lens[s])
    T = np.stack([g.permutation(V)[:4] for _ in range(V)]).astype(np.int32)
    decode(ngs, ctx, hist, lens, [1], 4, B, w, 3, 12, 4, 6, T)      # sequence 0 runs out of room after a step or two
    assert ctx.get_status() == ngs.STATUS_CAPACITY
