"""GPU parity on the degenerate and extreme shapes the C ABI accepts."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import dev_bf16, dev_i32
from test_gpu_head import TOL, check_table

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ngs():
    import paper_2411_03786_b200 as m
    return m


def test_empty_batches_are_accepted_and_launch_nothing(ngs):
    W = dev_bf16(synth.gaussian_weights(64, 64, 1.0, 1, "W"))
    ctx = ngs.SpecContext(W, W)
    lib = ngs.load_library()
    before = ctx.launch_count()
    h = ctx._h
    i32 = torch.zeros(4, dtype=torch.int32, device="cuda")
    p = C.c_void_p(i32.data_ptr())
    assert lib.verify_lmhead_argmax(h, C.c_void_p(W.data_ptr()), 0, p, None, None) == 0
    qs = (C.c_int * 1)(1)
    assert lib.draft_context_ngrams(h, p, p, 0, 4, qs, 1, 1, 1, 1, 0, p, p, None, None, None) == 0
    assert lib.accept_and_commit(h, p, p, p, 0, 1, 1, p, p, 4, p, p, p, None) == 0
    assert ctx.launch_count() == before
    # limits are enforced on the host
    assert lib.draft_context_ngrams(h, p, p, 1, 4, qs, 1, 1, 65, 1, 0, p, p, None, None, None) == -1      # B > 64
    assert lib.draft_context_ngrams(h, p, p, 1, 4, qs, 1, 1, 1, 17, 0, p, p, None, None, None) == -1      # w > 16
    assert lib.draft_context_ngrams(h, p, p, 1, 6, qs, 1, 1, 1, 1, 0, p, p, None, None, None) == -1       # cap % 4
    assert lib.draft_context_ngrams(h, p, p, 1, 4, qs, 1, 1, 1, 1, 2, p, p, None, None, None) == -4       # no table yet
    assert lib.verify_lmhead_argmax(h, C.c_void_p(W.data_ptr()), 65537, p, None, None) == -1
    ctx.close()


def test_largest_draft_shapes_match_the_oracle(ngs):
    V = 300
    W = dev_bf16(synth.gaussian_weights(V, 64, 1.0, 2, "W"))
    ctx = ngs.SpecContext(W, W)
    g = np.random.default_rng(3)
    T = np.stack([g.permutation(V)[:32] for _ in range(V)]).astype(np.int32)
    ctx.set_model_table(dev_i32(T))
    B, w, topk, qs = 64, 16, 64, [4, 3, 2, 1]
    S, cap = 5, 3000
    lens = np.array([3000, 2999, 17, 1, 0], np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, 3, lens[s])         # tiny alphabet: hundreds of candidate rows, many ties
    hist[1, :lens[1]] = g.integers(0, V, lens[1])
    for flags in (3, 2, 1):
        want = oracle.draft_batch(hist, lens, qs, topk, B, w, flags, T)
        got = ctx.draft_context_ngrams(dev_i32(hist), dev_i32(lens), qs, topk, B, w, flags)
        for a, b in zip(got, want):
            assert np.array_equal(a.cpu().numpy(), b)
    assert ctx.get_status() == 0
    ctx.close()


def test_widest_table_and_tiny_vocabulary(ngs):
    for V, d, k in ((40, 8, 32), (17, 16, 17), (2000, 72, 32)):
        E = synth.gaussian_weights(V, d, 1.0, V, "E")
        W = synth.gaussian_weights(V, d, 1.0, V, "W")
        ctx = ngs.SpecContext(dev_bf16(E), dev_bf16(W))
        tab, val, ext = ctx.build_model_ngram_tables(k, w_ext=16, with_values=True)
        check_table(tab.cpu().numpy(), val.cpu().numpy(), E, W, k, rows=None)
        assert np.array_equal(ext.cpu().numpy(), oracle.extend_table(tab.cpu().numpy(), 16))
        H = synth.hidden_literal(5, d, seed=V)
        am, mx = ctx.verify_lmhead_argmax(dev_bf16(H), with_max=True)
        ref_am, ref_mx, gap = oracle.verify(H, W)
        assert not ((am.cpu().numpy() != ref_am) & (gap >= TOL)).any()
        assert ctx.get_status() == 0
        ctx.close()


def test_maximum_verify_rows(ngs):
    V, d, M = 96, 64, 65536
    W = synth.gaussian_weights(V, d, 1.0, 5, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    H = synth.hidden_literal(M, d, seed=6)
    am, mx = ctx.verify_lmhead_argmax(dev_bf16(H), with_max=True)
    z = synth.bf16_bits_to_f32(H).astype(np.float64) @ synth.bf16_bits_to_f32(W).astype(np.float64).T
    ref = z.argmax(axis=1)
    srt = np.sort(z, axis=1)
    gap = srt[:, -1] - srt[:, -2]
    got = am.cpu().numpy()
    assert not ((got != ref) & (gap >= TOL)).any()
    assert np.abs(mx.cpu().numpy() - z.max(axis=1)).max() <= TOL
    rows = np.array([0, 127, 128, 65535])
    ref_am, _, _ = oracle.verify(H, W, rows=rows)           # the numpy shortcut above agrees with the oracle
    assert np.array_equal(ref[rows], ref_am)
    ctx.close()
