"""GPU parity for the integer stages (drafting, acceptance, commit): bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import dev_bf16, dev_i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ngs():
    import paper_2411_03786_b200 as m
    return m


@pytest.fixture(scope="module")
def small_ctx(ngs):
    V, d = 512, 64
    E = synth.gaussian_weights(V, d, 1.0, 1, "E")
    W = synth.gaussian_weights(V, d, 1.0, 1, "W")
    ctx = ngs.SpecContext(dev_bf16(E), dev_bf16(W))
    yield ctx
    ctx.close()


def random_table(V, k, seed):
    g = np.random.default_rng(seed)
    return np.stack([g.permutation(V)[:k] for _ in range(V)]).astype(np.int32)


def run_draft(ctx, hist, lens, qs, topk, B, w, flags, T, ext=None):
    if T is not None:
        ctx.set_model_table(dev_i32(T), dev_i32(ext) if ext is not None else None)
    out = ctx.draft_context_ngrams(dev_i32(hist), dev_i32(lens), qs, topk, B, w, flags)
    torch.cuda.synchronize()
    return [o.cpu().numpy() for o in out]


def assert_draft_equal(got, want):
    for g, w_, name in zip(got, want, ("drafts", "n_drafts", "src", "counts")):
        assert np.array_equal(g, w_), name


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4", "C5"])
def test_draft_matches_oracle_on_paper_shaped_histories(ngs, small_ctx, name):
    c = synth.config(name)
    V = 512                                    # token ids folded into the small context's vocabulary
    hist, lens, _ = synth.zipf_histories(c["S"], c["L"], c["V"], c["zipf"], c["copy"], c["seed"], cap=c["L"] + 64)
    hist = np.where(hist >= 0, hist % V, -1).astype(np.int32)
    T = random_table(V, c["k_tab"], 3)
    ext = oracle.extend_table(T, c["w"])
    for flags in (3, 1, 2, 0, 7):
        want = oracle.draft_batch(hist, lens, c["qs"], c["topk"], c["B"], c["w"], flags, T)
        assert_draft_equal(run_draft(small_ctx, hist, lens, c["qs"], c["topk"], c["B"], c["w"], flags, T), want)
        assert_draft_equal(run_draft(small_ctx, hist, lens, c["qs"], c["topk"], c["B"], c["w"], flags, T, ext), want)
    assert small_ctx.get_status() == 0


def test_draft_random_small_alphabets_and_ragged_lengths(ngs, small_ctx):
    g = np.random.default_rng(0)
    V = 512
    T = random_table(V, 5, 1)
    for trial in range(40):
        S = int(g.integers(1, 9))
        cap = int(g.integers(1, 80)) * 4
        A = int(g.integers(1, 6))
        lens = g.integers(0, cap + 1, S).astype(np.int32)
        hist = np.full((S, cap), -1, np.int32)
        for s in range(S):
            hist[s, :lens[s]] = g.integers(0, A, lens[s])
        n_q = int(g.integers(0, 5))
        qs = [int(q) for q in g.permutation([1, 2, 3, 4])[:n_q]]
        B = int(g.integers(1, 65)); w = int(g.integers(1, 17)); topk = int(g.integers(1, B + 1))
        flags = int(g.integers(0, 8)) | (oracle.flag_reserve(int(g.integers(0, B + 2))) if trial % 2 else 0)
        want = oracle.draft_batch(hist, lens, qs, topk, B, w, flags, T)
        assert_draft_equal(run_draft(small_ctx, hist, lens, qs, topk, B, w, flags, T), want)
    assert small_ctx.get_status() == 0


@pytest.mark.parametrize("L", [6000, 20000, 70000])      # history staged in shared memory / one CTA per sequence / a cluster of four
def test_draft_many_distinct_continuations_uses_the_exact_multi_pass_path(ngs, small_ctx, L):
    # q = 1 on a two-token-heavy history: thousands of distinct continuations, more than the
    # shared-memory table holds in one pass.
    g = np.random.default_rng(5)
    hist = g.integers(0, 512, (2, L)).astype(np.int32)
    hist[:, ::2] = 7                          # every other token is the query token
    hist[:, -1] = 7
    lens = np.array([L, L - 3], np.int32)
    hist[1, L - 4] = 7
    T = random_table(512, 4, 2)
    want = oracle.draft_batch(hist, lens, [1, 2], 6, 16, 4, 3, T)
    got = run_draft(small_ctx, hist, lens, [1, 2], 6, 16, 4, 3, T)
    assert_draft_equal(got, want)
    assert small_ctx.get_status() == 0


def test_draft_many_short_sequences(ngs, small_ctx):
    g = np.random.default_rng(8)
    S, cap, V = 700, 256, 512
    lens = g.integers(0, cap + 1, S).astype(np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, 6, lens[s]) if s % 2 else g.integers(0, V, lens[s])
    T = random_table(V, 6, 4)
    want = oracle.draft_batch(hist, lens, [3, 1], 5, 12, 6, 3, T)
    assert_draft_equal(run_draft(small_ctx, hist, lens, [3, 1], 5, 12, 6, 3, T), want)
    assert small_ctx.get_status() == 0


def test_draft_reports_bad_inputs_without_trapping(ngs, small_ctx):
    T = random_table(512, 4, 2)
    hist = np.zeros((2, 16), np.int32)
    hist[0, :8] = [1, 2, 3, 1, 2, 3, 1, 999]      # last token outside the vocabulary: no model rows
    hist[1, :8] = [1, 2, 3, 1, 2, 3, 1, 2]
    lens = np.array([8, 40], np.int32)            # second length exceeds cap
    drafts, nd, src, cnt = run_draft(small_ctx, hist, lens, [1], 2, 4, 2, 3, T)
    st = small_ctx.get_status()
    assert st & ngs.STATUS_TOKEN_RANGE and st & ngs.STATUS_CAPACITY
    assert nd[1] == 0 and (drafts[1] == -1).all()
    assert (src[0] != 0).all()
    assert small_ctx.get_status() == 0            # reading clears the bits


@pytest.mark.parametrize("S,B,w", [(1, 4, 4), (64, 16, 8), (5, 64, 16), (1000, 33, 1)])
def test_accept_commit_matches_oracle(ngs, small_ctx, S, B, w):
    g = np.random.default_rng(S + B + w)
    A = 3
    drafts = g.integers(0, A, (S, B, w)).astype(np.int32)
    P = g.integers(0, A, (S, B, w + 1)).astype(np.int32)
    for s in range(0, S, 3):                       # plant longer accepted prefixes
        b = int(g.integers(0, B)); a = int(g.integers(0, w + 1))
        P[s, b, :a] = drafts[s, b, :a]
    nd = g.integers(0, B + 1, S).astype(np.int32)
    cap = 40
    lens = g.integers(0, cap + 1, S).astype(np.int32)
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, A, lens[s])
    h_ref, l_ref = hist.copy(), lens.copy()
    acc_r, best_r, com_r = oracle.accept_commit(drafts, nd, P, h_ref, l_ref)
    dh, dl = dev_i32(hist), dev_i32(lens)
    acc, best, com = small_ctx.accept_and_commit(dev_i32(drafts), dev_i32(nd), dev_i32(P), dh, dl)
    assert np.array_equal(acc.cpu().numpy(), acc_r) and np.array_equal(best.cpu().numpy(), best_r)
    assert np.array_equal(com.cpu().numpy(), com_r)
    assert np.array_equal(dh.cpu().numpy(), h_ref) and np.array_equal(dl.cpu().numpy(), l_ref)
    st = small_ctx.get_status()
    assert bool(st & ngs.STATUS_CAPACITY) == bool((acc_r < 0).any())


def test_toy_model_decode_is_lossless_and_fully_accepted(ngs):
    """End to end on the Tiny configuration: table build -> (draft -> verify -> accept) x steps."""
    c = synth.config("C1")
    E = synth.gaussian_weights(c["V"], c["d"], c["wstd"], 0, "E", "f32")
    W = synth.gaussian_weights(c["V"], c["d"], c["wstd"], 0, "W", "f32")
    Wb = oracle.round_to_bf16(W)
    Hall = synth.unit_rows_bf16(E)
    hist0, lens0, _ = synth.zipf_histories(1, c["L"], c["V"], c["zipf"], c["copy"], 0, cap=c["L"] + 256)
    prompt = hist0[0, :lens0[0]]
    n = 60
    ref = oracle.toy_greedy(prompt[-1], n, Hall, Wb)
    ctx = ngs.SpecContext(torch.from_numpy(E).cuda(), torch.from_numpy(W).cuda())
    dHall = dev_bf16(Hall)
    tab, _, _ = ctx.build_model_ngram_tables(c["k_tab"], rows=dHall, w_ext=c["w"])
    T_ref, _ = oracle.model_table(Hall, Wb, c["k_tab"])
    assert np.array_equal(tab.cpu().numpy(), T_ref)
    for qs, expect_full in ((c["qs"], False), ((), True)):
        hist, lens = dev_i32(hist0), dev_i32(lens0)
        accs = []
        while int(lens[0]) - len(prompt) < n:
            drafts, nd, _, _ = ctx.draft_context_ngrams(hist, lens, qs, c["topk"], c["B"], c["w"])
            L = int(lens[0])
            block = torch.cat([hist[:, L - 1:L].expand(c["B"], 1), drafts[0].clamp(min=0)], dim=1)   # [B, w+1]
            H = dHall[block.reshape(-1).long()].contiguous()
            am, _ = ctx.verify_lmhead_argmax(H)
            acc, best, _ = ctx.accept_and_commit(drafts, nd, am.view(1, c["B"], c["w"] + 1), hist, lens)
            accs.append(int(acc[0]))
        gen = hist[0, len(prompt):len(prompt) + n].cpu().tolist()
        assert gen == ref
        if expect_full:
            assert accs == [c["w"]] * len(accs)
        g2, a2, _ = oracle.toy_speculative(prompt, n, Hall, Wb, T_ref, list(qs), c["topk"], c["B"], c["w"])
        assert accs == a2
    assert ctx.get_status() == 0
    ctx.close()


@pytest.mark.parametrize("S,B,w", [(1, 8, 5), (7, 4, 3), (64, 16, 8), (300, 2, 2), (5, 8, 4)])
def test_fused_verify_accept_equals_the_two_calls_and_the_oracle(ngs, S, B, w):
    V, d = 777, 96
    g = np.random.default_rng(S * 100 + B)
    W = synth.gaussian_weights(V, d, 1.0, 3, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    M = S * B * (w + 1)
    drafts = g.integers(0, V, (S, B, w)).astype(np.int32)
    nd = g.integers(0, B + 1, S).astype(np.int32)
    targets = g.integers(0, V, (S, B, w + 1)).astype(np.int32)
    for s in range(S):                                  # plant accepted prefixes of random length
        b, a = int(g.integers(0, B)), int(g.integers(0, w + 1))
        targets[s, b, :a] = drafts[s, b, :a]
    H = synth.hidden_planted(W, targets.reshape(-1), seed=S, gain=24.0)
    cap = 32
    lens = g.integers(0, cap - 2, S).astype(np.int32)
    lens[0] = cap - 1                                   # too full for more than one token
    hist = np.full((S, cap), -1, np.int32)
    for s in range(S):
        hist[s, :lens[s]] = g.integers(0, V, lens[s])
    dH, dD, dN = dev_bf16(H), dev_i32(drafts), dev_i32(nd)
    h1, l1 = dev_i32(hist), dev_i32(lens)
    am, _ = ctx.verify_lmhead_argmax(dH)
    acc1, best1, com1 = ctx.accept_and_commit(dD, dN, am.view(S, B, w + 1), h1, l1)
    h2, l2 = dev_i32(hist), dev_i32(lens)
    am2, acc2, best2, com2 = ctx.verify_accept_commit(dH, dD, dN, h2, l2)
    assert torch.equal(am2.reshape(-1), am) and np.array_equal(am.cpu().numpy(), targets.reshape(-1))
    for a, b in ((acc1, acc2), (best1, best2), (com1, com2), (h1, h2), (l1, l2)):
        assert torch.equal(a, b)
    h_ref, l_ref = hist.copy(), lens.copy()
    acc_r, best_r, com_r = oracle.accept_commit(drafts, nd, targets, h_ref, l_ref)
    assert np.array_equal(acc2.cpu().numpy(), acc_r) and np.array_equal(best2.cpu().numpy(), best_r)
    assert np.array_equal(com2.cpu().numpy(), com_r) and np.array_equal(h2.cpu().numpy(), h_ref)
    assert np.array_equal(l2.cpu().numpy(), l_ref)
    # small outputs may live in mapped pinned host memory: the kernel's stores are the device-to-host transfer
    pin = lambda *shape: torch.full(shape, -9, dtype=torch.int32).pin_memory()
    out3 = (pin(S), pin(S), pin(S, w + 1))
    h3, l3 = dev_i32(hist), dev_i32(lens)
    ctx.verify_accept_commit(dH, dD, dN, h3, l3, out=out3)
    torch.cuda.synchronize()
    assert np.array_equal(out3[0].numpy(), acc_r) and np.array_equal(out3[1].numpy(), best_r)
    assert np.array_equal(out3[2].numpy(), com_r) and np.array_equal(h3.cpu().numpy(), h_ref)
    ctx.get_status()
    ctx.close()


def test_ablation_counters_match_oracle(ngs, small_ctx):
    g = np.random.default_rng(12)
    S, B, w = 500, 10, 6
    src = g.integers(-1, 5, (S, B)).astype(np.int32)
    acc = g.integers(-1, w + 1, S).astype(np.int32)
    best = np.where(acc >= 0, g.integers(0, B, S), -1).astype(np.int32)
    want = oracle.accumulate_stats(acc, best, src, w)
    want = oracle.accumulate_stats(acc, best, src, w, stats=want)
    st = small_ctx.accumulate_stats(dev_i32(acc), dev_i32(best), dev_i32(src), w)
    st = small_ctx.accumulate_stats(dev_i32(acc), dev_i32(best), dev_i32(src), w, stats=st)
    assert np.array_equal(st.cpu().numpy(), want)
