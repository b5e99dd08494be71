import numpy as np

import synth


def test_streams_are_reproducible_and_independent():
    a = synth.stream(3, "E").random(8)
    b = synth.stream(3, "E").random(8)
    c = synth.stream(3, "W").random(8)
    assert np.array_equal(a, b) and not np.array_equal(a, c)


def test_bf16_roundtrip_matches_torch():
    import torch
    x = synth.stream(0, "x").standard_normal(4096, dtype=np.float32)
    x[:4] = np.array([1.00390625, 1.01171875, -1.00390625, 3.0e-39], dtype=np.float32)  # exact ties, subnormal
    bits = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    assert np.array_equal(synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(bits)), bits)


def test_histories_shape_and_copy_fraction():
    h, l, f = synth.zipf_histories(3, 2048, 32000, 1.1, 0.30, seed=2, cap=2050)
    assert h.shape == (3, 2052) and h.dtype == np.int32 and (l == 2048).all()
    assert (h[:, :2048] >= 0).all() and (h[:, :2048] < 32000).all() and (h[:, 2048:] == -1).all()
    assert 0.2 < f < 0.4
    h2, _, _ = synth.zipf_histories(3, 2048, 32000, 1.1, 0.30, seed=2, cap=2050)
    assert np.array_equal(h, h2)
    # the most frequent token is a few per cent of positions (heavy Zipf head)
    _, c = np.unique(h[0, :2048], return_counts=True)
    assert 0.03 < c.max() / 2048 < 0.25


def test_planted_targets_follow_the_recipe():
    S, B, w, V = 5, 4, 3, 100
    g = synth.stream(1, "d")
    drafts = g.integers(0, V, (S, B, w)).astype(np.int32)
    nd = np.array([4, 2, 0, 1, 4], dtype=np.int32)
    t, rows, acc = synth.planted_targets(drafts, nd, None, V, 1.1, 0.55, seed=7)
    for s in range(S):
        if nd[s] == 0:
            continue
        r, a = rows[s], acc[s]
        assert r < nd[s] and 0 <= a <= w
        assert (t[s, r, :a] == drafts[s, r, :a]).all()
        if a < w:
            assert t[s, r, a] != drafts[s, r, a]
