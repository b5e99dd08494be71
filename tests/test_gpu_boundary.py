"""GPU checks of the boundary's failure and housekeeping paths: a bounded device-side wait that runs out
(in the allowed form: a barrier nobody arrives at, a limit of microseconds), an incomplete verification,
the table built in slices, a freshly quantised 8-bit head read without a host synchronisation, and a
corrupt history token."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import dev_bf16, dev_i32

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def ngs():
    import paper_2411_03786_b200 as m
    return m


def test_a_bounded_wait_that_runs_out_sets_the_status_and_leaves_the_context_usable(ngs):
    V, d, M = 4136, 320, 77
    W = synth.gaussian_weights(V, d, d ** -0.5, 41, "W")
    H = synth.hidden_literal(M, d, seed=42)
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    ref_am, _, gap = oracle.verify(H, W)
    ctx.debug_expire_wait(limit_ns=20_000)                  # nobody arrives at the barrier: the wait gives up
    assert ctx.get_status() == ngs.STATUS_TIMEOUT
    assert ctx.get_status() == 0                            # read and cleared
    am, mx = ctx.verify_lmhead_argmax(dev_bf16(H), with_max=True)     # the context works as before
    bad = am.cpu().numpy() != ref_am
    assert not (bad & (gap >= TOL)).any() and ctx.get_status() == 0
    # a contraction CTA that gave up: the next verification must not pass partial arg maxima for results
    ctx.debug_expire_wait(limit_ns=20_000, mark_verify_incomplete=True)
    am2, mx2 = ctx.verify_lmhead_argmax(dev_bf16(H), with_max=True)
    assert (am2 == -1).all() and torch.isinf(mx2).all() and (mx2 < 0).all()
    assert ctx.get_status() == ngs.STATUS_TIMEOUT
    keys = ctx.verify_lmhead_keys(dev_bf16(H), 0)           # and the one after that is complete again
    am3, _ = ngs.unpack_keys(keys, V)
    assert torch.equal(am3, am) and ctx.get_status() == 0
    # same for the fused call: nothing is accepted or committed from an incomplete verification
    S, B, w = 1, 7, 10
    hist_h, lens_h, _ = synth.zipf_histories(S, 300, V, 1.1, 0.3, seed=43, cap=320)
    hist, lens = dev_i32(hist_h), dev_i32(lens_h)
    drafts, nd, _, _ = ctx.draft_context_ngrams(hist, lens, [1], B, B, w, flags=ngs.FLAG_DEDUP)
    ctx.debug_expire_wait(limit_ns=20_000, mark_verify_incomplete=True)
    acc = torch.full((S,), -7, dtype=torch.int32, device="cuda")
    out = (acc, torch.full((S,), -7, dtype=torch.int32, device="cuda"), torch.full((S, w + 1), -7, dtype=torch.int32, device="cuda"))
    P, _, _, _ = ctx.verify_accept_commit(dev_bf16(H), drafts, nd, hist, lens, out=out)
    assert (P == -1).all() and int(acc[0]) == -7 and torch.equal(lens.cpu(), torch.from_numpy(lens_h))
    assert ctx.get_status() == ngs.STATUS_TIMEOUT
    ctx.close()


@pytest.mark.parametrize("V,d,k", [(1000, 200, 8), (4136, 64, 10), (300, 64, 32)])
def test_table_built_in_two_slices_equals_the_whole_build(ngs, V, d, k):
    from paper_2411_03786_b200 import multigpu
    E = synth.gaussian_weights(V, d, 1.0, 7 * V + d, "E")
    W = synth.gaussian_weights(V, d, 1.0, 7 * V + d, "W")
    ctx = ngs.SpecContext(dev_bf16(E), dev_bf16(W))
    whole, val, ext = ctx.build_model_ngram_tables(k, w_ext=4, with_values=True)
    tab = torch.full((V, k), -9, dtype=torch.int32, device="cuda")
    vals = torch.zeros((V, k), dtype=torch.float32, device="cuda")
    for rank in range(2):                                   # what two ranks would each build
        first, count = multigpu.shard_sequences(V, rank, 2)
        ctx.build_model_ngram_table_rows(k, first, count, tab, val=vals)
        if rank == 0:
            assert (tab[count:] == -9).all()                # a slice call writes its own rows only
    assert torch.equal(tab, whole) and torch.equal(vals, val)
    assert torch.equal(ctx.extend_model_table(tab, 4), ext)
    # ragged slices, down to one row and an empty one; rows given by the caller
    rows = synth.hidden_literal(V, d, seed=5)
    whole2, _, _ = ctx.build_model_ngram_tables(k, rows=dev_bf16(rows))
    tab2 = torch.full((V, k), -9, dtype=torch.int32, device="cuda")
    cuts = [0, 1, 1, 130, V // 2 + 3, V]
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        ctx.build_model_ngram_table_rows(k, lo, hi - lo, tab2, rows=dev_bf16(rows))
    assert torch.equal(tab2, whole2)
    t1, e1 = multigpu.sharded_table_build(ctx, k, 4, rank=0, world=1)          # one rank, no process group
    assert torch.equal(t1, whole) and torch.equal(e1, ext)
    with pytest.raises(ngs.SpecError, match="not inside"):
        ctx.build_model_ngram_table_rows(k, V - 3, 4, tab)
    assert ctx.get_status() == 0
    ctx.close()


def test_fresh_8bit_head_is_read_correctly_without_a_host_synchronisation(ngs):
    """The head quantisation lets the next kernel start early; the verification that follows on the same
    stream must still see the finished codes (it may not fetch weights before its dependency wait)."""
    V, d, M = 40000, 1024, 48
    W = synth.gaussian_weights(V, d, d ** -0.5, 51, "W")
    H = synth.hidden_literal(M, d, seed=52)
    Wq, Ws = oracle.quantize_rows_e4m3(W)
    Hq, Hs = oracle.quantize_rows_e4m3(H)
    ref_am, ref_mx, gap = oracle.verify_q8(Hq, Hs, Wq, Ws)
    dW, dH = dev_bf16(W), dev_bf16(H)
    ctx = ngs.SpecContext(dW, dW)
    scratch = ctx.quantize_rows_fp8(dH)
    torch.cuda.synchronize()
    for rep in range(3):
        wq, ws = ctx.quantize_head_fp8()                     # fresh buffers every time, no synchronisation after it
        am, mx = ctx.verify_lmhead_argmax_fp8(None, scratch=scratch, with_max=True)
        am, mx = am.cpu().numpy(), mx.cpu().numpy().astype(np.float64)
        bad = am != ref_am
        assert not (bad & (gap >= TOL)).any() and np.abs(mx - ref_mx).max() <= TOL
    assert ctx.get_status() == 0
    ctx.close()


def test_context_row_with_a_corrupt_token_is_dropped_and_reported(ngs):
    V, d = 64, 64
    W = synth.gaussian_weights(V, d, 1.0, 61, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    tab, _, _ = ctx.build_model_ngram_tables(4, w_ext=3)
    T = tab.cpu().numpy()
    g = np.random.default_rng(62)
    S, L, cap = 6, 120, 128
    hist_h = np.full((S, cap), -1, np.int32)
    hist_h[:, :L] = g.integers(0, 6, (S, L))
    hist_h[:, 111:113] = hist_h[:, L - 2:L]                 # a recent occurrence of the last two tokens ...
    hist_h[:, 115] = V + 5                                  # ... whose continuation holds a corrupt token: too large,
    hist_h[1::2, 114] = -3                                  # or negative
    lens_h = np.full(S, L, np.int32)
    for flags in (3, 1, 2, 3 | ngs.flag_reserve(2)):
        got = ctx.draft_context_ngrams(dev_i32(hist_h), dev_i32(lens_h), [2, 1], 16, 24, 3, flags=flags)
        want = oracle.draft_batch(hist_h, lens_h, [2, 1], 16, 24, 3, flags, T)
        for a, b in zip(got, want):
            assert np.array_equal(a.cpu().numpy(), b)
        dr = got[0].cpu().numpy()
        assert ((dr >= -1) & (dr < V)).all()
        assert ctx.get_status() == ngs.STATUS_TOKEN_RANGE
    ctx.close()
