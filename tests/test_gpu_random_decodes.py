"""GPU parity over seeded random decode loops and acceptance batches: every shape parameter is drawn at random
(sequences, history lengths from empty to thousands of tokens, alphabets from 2 symbols to the vocabulary, query
lengths, widths, flags), the indexed drafting and the indexed commit are compared with the oracle at every step."""
import numpy as np
import pytest

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


def random_histories(g, S, Lmax, alpha, extra):
    """Ragged histories over `alpha` symbols with copied spans; `extra` free slots behind the longest one."""
    cap = (Lmax + extra + 3) // 4 * 4
    lens = np.array([Lmax if s == 0 else int(g.integers(0, Lmax + 1)) for s in range(S)], np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        h = g.integers(0, alpha, lens[s])
        if g.random() < 0.6 and lens[s] > 40:
            for _ in range(int(lens[s]) // 50):
                a, b, n = int(g.integers(0, lens[s] - 20)), int(g.integers(0, lens[s] - 20)), int(g.integers(4, 20))
                h[b:b + n] = h[a:a + n]
        hist[s, :lens[s]] = h
    return hist, lens


@pytest.mark.parametrize("seed", range(40))
def test_random_indexed_decode(ngs, ctx, seed):
    g = np.random.default_rng(770000 + seed)
    S = int(g.integers(1, 12))
    Lmax = int(g.choice([0, 5, 40, 300, 2000, 9000]))
    alpha = int(g.choice([2, 3, 6, 40, V]))
    steps = int(g.integers(5, 40))
    w, B, k_tab = int(g.integers(1, 9)), int(g.integers(1, 17)), int(g.integers(1, 9))
    topk = int(g.integers(1, B + 1))
    qs = [int(q) for q in g.choice([1, 2, 3, 4], int(g.integers(1, 4)), replace=False)]
    flags = int(g.choice([1, 2, 3, 7, 5]))
    hist_h, lens_h = random_histories(g, S, Lmax, alpha, steps * (w + 1) + 8)
    hist, lens = dev_i32(hist_h), dev_i32(lens_h)
    T = np.stack([g.permutation(V)[:k_tab] for _ in range(V)]).astype(np.int32)
    ctx.set_model_table(dev_i32(T), dev_i32(oracle.extend_table(T, w)))
    index = ctx.context_index_build(hist, lens, qs, w, flags & ngs.FLAG_KEY_NEXT_TOKEN)
    for step in range(steps):
        want = oracle.draft_batch(hist_h, lens_h, qs, topk, B, w, flags, T)
        got = ctx.draft_context_ngrams_indexed(index, hist, lens, qs, topk, B, w, flags)
        for a, b, name in zip(got, want, ("drafts", "n_drafts", "src", "counts")):
            assert np.array_equal(a.cpu().numpy(), b), f"step {step}: {name}"
        P = g.integers(0, alpha, (S, B, w + 1)).astype(np.int32)   # accept a random prefix of a random row
        for s in range(S):
            if want[1][s] > 0:
                b, a = int(g.integers(0, want[1][s])), int(g.integers(0, w + 1))
                P[s, b, :a] = want[0][s, b, :a]
        acc_r, best_r, com_r = oracle.accept_commit(want[0], want[1], P, hist_h, lens_h)
        acc, best, com = ctx.accept_and_commit_indexed(index, got[0], got[1], dev_i32(P), hist, lens)
        assert np.array_equal(acc.cpu().numpy(), acc_r) and np.array_equal(best.cpu().numpy(), best_r)
        assert np.array_equal(com.cpu().numpy(), com_r) and np.array_equal(lens.cpu().numpy(), lens_h)
    assert np.array_equal(hist.cpu().numpy(), hist_h)
    assert ctx.get_status() == 0


@pytest.mark.parametrize("seed", range(40))
def test_random_acceptance_batch(ctx, seed):
    g = np.random.default_rng(880000 + seed)
    S = int(g.choice([1, 3, 64, 700, 5000]))
    B, w, alpha = int(g.integers(1, 65)), int(g.integers(1, 17)), int(g.choice([2, 5, 1000]))
    cap = int(g.integers(1, 12)) * 4                                # short capacities: some commits do not fit
    drafts = g.integers(0, alpha, (S, B, w)).astype(np.int32)
    nd = g.integers(0, B + 1, S).astype(np.int32)
    P = g.integers(0, alpha, (S, B, w + 1)).astype(np.int32)
    P[:, :, :w] = np.where(g.random((S, B, w)) < 0.8, drafts, P[:, :, :w])   # long accepted prefixes
    lens = g.integers(0, cap + 1, S).astype(np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, alpha, lens[s])
    hist_h, lens_h = hist.copy(), lens.copy()
    acc_r, best_r, com_r = oracle.accept_commit(drafts, nd, P, hist_h, lens_h)
    dh, dl = dev_i32(hist), dev_i32(lens)
    acc, best, com = ctx.accept_and_commit(dev_i32(drafts), dev_i32(nd), dev_i32(P), dh, dl)
    assert np.array_equal(acc.cpu().numpy(), acc_r) and np.array_equal(best.cpu().numpy(), best_r)
    assert np.array_equal(com.cpu().numpy(), com_r)
    assert np.array_equal(dl.cpu().numpy(), lens_h) and np.array_equal(dh.cpu().numpy(), hist_h)
    ctx.get_status()                                                # capacity bits are expected here: clear them
