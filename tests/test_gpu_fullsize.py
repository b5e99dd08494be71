"""GPU parity at the full benchmark sizes (configs C2-C5), in the launch configuration bench.py times.

The oracle cannot afford the whole contractions here: the verification of C2 is compared on all 48 rows,
everything else on at least 512 sampled rows (first and last row of the first, a middle and the last tile
of every tile group, plus seeded random rows); integer stages are compared in full.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import dev_bf16, dev_i32, weights
from test_gpu_head import TOL, check_table

pytestmark = pytest.mark.gpu
RHO = 0.55


@pytest.fixture(scope="module")
def heads():
    """One context (and one model table) per distinct head: C2/C3 share one, C4/C5 the other."""
    import paper_2411_03786_b200 as ngs
    cache = {}

    def get(name):
        c = synth.config(name)
        key = (c["V"], c["d"], c["wseed"])
        if key not in cache:
            E, W = weights(c, "E"), weights(c, "W")
            ctx = ngs.SpecContext(dev_bf16(E), dev_bf16(W))
            k = 10 if c["V"] > 100000 else 8
            tab, val, ext = ctx.build_model_ngram_tables(k, w_ext=10, with_values=True)
            torch.cuda.synchronize()
            cache[key] = dict(E=E, W=W, ctx=ctx, tab=tab, val=val, ext=ext, k=k)
        return c, cache[key]

    yield get
    for h in cache.values():
        h["ctx"].close()


N_SAMPLE = 512      # rows the oracle checks wherever it cannot afford all of them


def sample_rows(n_rows, n, seed, tile=128, group=1):
    """At least ``n`` distinct rows (all of them when there are no more): the first and last row of the
    first, a middle and the last 128-row tile of every group of ``group`` tiles (the contraction walks the
    rows in such groups; the last group and the last tile are ragged), then seeded random rows."""
    if n_rows <= n:
        return np.arange(n_rows, dtype=np.int64)
    n_tiles = (n_rows + tile - 1) // tile
    rows = {0, 1, n_rows - 1, n_rows - 2}
    for g0 in range(0, n_tiles, group):
        g1 = min(n_tiles, g0 + group)
        for t in {g0, (g0 + g1 - 1) // 2, g1 - 1}:
            rows |= {t * tile, min(n_rows, (t + 1) * tile) - 1}
    g = np.random.default_rng(seed)
    while len(rows) < n:
        rows |= set(g.integers(0, n_rows, n - len(rows)).tolist())
    return np.array(sorted(rows), dtype=np.int64)


@pytest.mark.parametrize("name", ["C2", "C4"])
def test_model_table_sampled_rows(heads, name):
    c, h = heads(name)
    V = c["V"]
    tab = h["tab"].cpu().numpy()
    # the table kernel runs its 128-row tiles in groups of 16 at these sizes; add rows whose best column lies in
    # the first / last 256 columns of the vocabulary (the first and last chunk a CTA sweeps)
    rows = set(sample_rows(V, N_SAMPLE, seed=c["seed"], group=16).tolist())
    rows |= set(np.flatnonzero(tab[:, 0] < 256)[:16].tolist()) | set(np.flatnonzero(tab[:, 0] >= V - 256)[:16].tolist())
    rows = np.array(sorted(rows), dtype=np.int64)
    assert len(rows) >= N_SAMPLE
    frac = check_table(tab, h["val"].cpu().numpy(), h["E"], h["W"], h["k"], rows=rows)
    print(f"{name} table: {round(frac * len(rows))} of {len(rows)} sampled rows have the oracle's top-{h['k']} list exactly")
    assert frac >= 0.9
    assert tab.min() >= 0 and tab.max() < V
    # extended table: integer stage, exact given the table (all rows)
    ext = h["ext"].cpu().numpy()
    ref = oracle.extend_table(tab, 10)
    assert np.array_equal(ext, ref)


def test_model_unigram_sampled_rows_at_full_size(heads):
    c, h = heads("C2")
    idx, dist2 = h["ctx"].build_model_unigram(25)
    dist2 = dist2.cpu().numpy().astype(np.float64)
    rows = sample_rows(c["V"], N_SAMPLE, seed=11, group=16)
    ref = oracle.unigram_dist2(h["W"], h["E"], rows=rows)
    assert np.abs(dist2[rows] - ref).max() <= 2e-3 * ref.max()
    assert np.array_equal(idx.cpu().numpy(), oracle.smallest_k(dist2, 25))       # integer stage: exact
    assert np.isfinite(dist2).all() and (dist2 >= 0).all()


@pytest.mark.parametrize("name", ["C2", "C3", "C4", "C5"])
def test_whole_step_at_full_size(heads, name):
    c, h = heads(name)
    ctx = h["ctx"]
    S, B, w, M = c["S"], c["B"], c["w"], c["M"]
    hist_h, lens_h, _ = synth.zipf_histories(S, c["L"], c["V"], c["zipf"], c["copy"], c["seed"], cap=c["L"] + 64)
    T = h["tab"].cpu().numpy()
    hist, lens = dev_i32(hist_h), dev_i32(lens_h)
    # drafting: bit-exact against the oracle given the same table
    drafts, nd, src, cnt = ctx.draft_context_ngrams(hist, lens, c["qs"], c["topk"], B, w)
    want = oracle.draft_batch(hist_h, lens_h, c["qs"], c["topk"], B, w, 3, T)
    for got, exp in zip((drafts, nd, src, cnt), want):
        assert np.array_equal(got.cpu().numpy(), exp)
    # verification on planted and on literal hidden states: sampled rows against the oracle
    targets, _, planted_a = synth.planted_targets(want[0], want[1], None, c["V"], c["zipf"], RHO, seed=c["seed"])
    for kind in ("planted", "literal"):
        H = synth.hidden_planted(h["W"], targets.reshape(-1), seed=c["seed"]) if kind == "planted" else \
            synth.hidden_literal(M, c["d"], seed=c["seed"])
        am, mx = ctx.verify_lmhead_argmax(dev_bf16(H), with_max=True)
        am_h, mx_h = am.cpu().numpy(), mx.cpu().numpy().astype(np.float64)
        # literal hidden states: all M rows when M <= 512 (C2: all 48), else >= 512 rows with the first and last
        # row of every 128-row tile class; planted ones are also compared with their targets in full below
        rows = sample_rows(M, N_SAMPLE if kind == "literal" else 64, seed=7)
        ref_am, ref_mx, gap = oracle.verify(H, h["W"], rows=rows)
        bad = am_h[rows] != ref_am
        assert not (bad & (gap >= TOL)).any()
        assert np.abs(mx_h[rows] - ref_mx).max() <= TOL
        print(f"{name} {kind}: {len(rows)} of {M} rows against the oracle, {int(bad.sum())} differ (all inside the tie margin), "
              f"max |logit error| {np.abs(mx_h[rows] - ref_mx).max():.2e}")
        assert am_h.min() >= 0 and am_h.max() < c["V"]
        if kind == "planted":
            assert np.array_equal(am_h, targets.reshape(-1))        # margins are wide by construction
            # acceptance and commit: bit-exact, and the planted accepted lengths come back
            h_ref, l_ref = hist_h.copy(), lens_h.copy()
            acc_r, best_r, com_r = oracle.accept_commit(want[0], want[1], am_h.reshape(S, B, w + 1), h_ref, l_ref)
            acc, best, com = ctx.accept_and_commit(drafts, nd, am.view(S, B, w + 1), hist, lens)
            assert np.array_equal(acc.cpu().numpy(), acc_r) and np.array_equal(best.cpu().numpy(), best_r)
            assert np.array_equal(com.cpu().numpy(), com_r)
            assert np.array_equal(hist.cpu().numpy(), h_ref) and np.array_equal(lens.cpu().numpy(), l_ref)
            has = want[1] > 0
            assert (acc_r[has] >= planted_a[has]).all()
    assert ctx.get_status() == 0
