"""Whole-step invariants on the toy model (hidden state = unit-length embedding of the last token).

Speculative decoding with greedy verification is lossless: whatever the drafts, the
tokens equal plain greedy decoding.  With model-bigram drafts built from the same
matrix, the rank-0 chain is the greedy continuation itself, so every drafted token
is accepted.
"""
import numpy as np

import oracle
import synth


def toy(seed=0):
    c = synth.config("C1")
    E = synth.gaussian_weights(c["V"], c["d"], c["wstd"], seed, "E", "f32")
    W = oracle.round_to_bf16(synth.gaussian_weights(c["V"], c["d"], c["wstd"], seed, "W", "f32"))
    Hall = synth.unit_rows_bf16(E)
    T, _ = oracle.model_table(Hall, W, c["k_tab"])
    hist, lens, _ = synth.zipf_histories(1, c["L"], c["V"], c["zipf"], c["copy"], seed)
    return c, Hall, W, T, hist[0, :lens[0]]


def test_mixed_drafts_are_lossless():
    c, Hall, W, T, prompt = toy()
    n = 60
    ref = oracle.toy_greedy(prompt[-1], n, Hall, W)
    gen, accs, _ = oracle.toy_speculative(prompt, n, Hall, W, T, c["qs"], c["topk"], c["B"], c["w"])
    assert gen == ref
    assert all(0 <= a <= c["w"] for a in accs)


def test_model_bigram_draft_is_accepted_at_every_position():
    c, Hall, W, T, prompt = toy()
    n = 40
    ref = oracle.toy_greedy(prompt[-1], n, Hall, W)
    gen, accs, bests = oracle.toy_speculative(prompt, n, Hall, W, T, [], c["topk"], c["B"], c["w"])
    assert gen == ref
    assert accs == [c["w"]] * len(accs) and bests == [0] * len(bests)
    assert len(accs) == -(-n // (c["w"] + 1))          # w+1 tokens per call


def test_random_drafts_are_lossless_too():
    c, Hall, W, T, prompt = toy(seed=0)
    g = np.random.default_rng(1)
    n = 25
    ref = oracle.toy_greedy(prompt[-1], n, Hall, W)

    def random_drafts(step, hist, L):
        d = g.integers(0, c["V"], (1, c["B"], c["w"])).astype(np.int32)
        if step % 2 == 0:                 # sometimes plant a correct first token
            d[0, 2, 0] = ref[L - len(prompt)] if L - len(prompt) < n else 0
        return d, np.array([c["B"]], np.int32)

    gen, accs, _ = oracle.toy_speculative(prompt, n, Hall, W, None, [], 1, c["B"], c["w"],
                                          drafts_override=random_drafts)
    assert gen == ref and max(accs) >= 1
