"""GPU parity at the full benchmark sizes (configs C2-C5), in the launch configuration bench.py times.

The oracle cannot afford the whole contractions here, so rows are sampled (first and last rows of the
first and last tiles, plus seeded random rows); integer stages are compared in full.
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


def sample_rows(n_rows, n, seed, tile=128):
    edge = {0, 1, tile - 1, tile, n_rows - 1, max(0, n_rows - 2), (n_rows - 1) // tile * tile}
    g = np.random.default_rng(seed)
    rows = sorted({r for r in edge if 0 <= r < n_rows} | set(g.integers(0, n_rows, n).tolist()))
    return np.array(rows, dtype=np.int64)


@pytest.mark.parametrize("name", ["C2", "C4"])
def test_model_table_sampled_rows(heads, name):
    c, h = heads(name)
    rows = sample_rows(c["V"], 12, seed=c["seed"])
    frac = check_table(h["tab"].cpu().numpy(), h["val"].cpu().numpy(), h["E"], h["W"], h["k"], rows=rows)
    assert frac >= 0.9
    tab = h["tab"].cpu().numpy()
    assert tab.min() >= 0 and tab.max() < c["V"]
    # extended table: integer stage, exact given the table
    ext = h["ext"].cpu().numpy()
    sel = sample_rows(c["V"], 200, seed=1)
    ref = oracle.extend_table(tab, 10)
    assert np.array_equal(ext[sel], ref[sel])


def test_model_unigram_sampled_rows_at_full_size(heads):
    c, h = heads("C2")
    idx, dist2 = h["ctx"].build_model_unigram(25)
    dist2 = dist2.cpu().numpy().astype(np.float64)
    rows = sample_rows(c["V"], 12, seed=11)
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
        rows = sample_rows(M, 12, seed=7)
        ref_am, ref_mx, gap = oracle.verify(H, h["W"], rows=rows)
        bad = am_h[rows] != ref_am
        assert not (bad & (gap >= TOL)).any()
        assert np.abs(mx_h[rows] - ref_mx).max() <= TOL
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
