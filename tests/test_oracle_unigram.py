"""Pins for the oracle's model unigram (Section 4.1 "Unigram")."""
import numpy as np

import oracle
import synth


def f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def centred(W):
    w = f64(W)
    return f64(synth.f32_to_bf16_bits((w - w.mean(axis=0)).astype(np.float32)))


def test_gram_matrix_identity():
    # sum_y (a . v_y)^2 = a^T (E^T E) a: the d x d covariance form of the same distance
    W = synth.gaussian_weights(150, 48, 1.0, 1, "W")
    E = synth.gaussian_weights(150, 48, 1.0, 1, "E")
    c = centred(W)
    G = f64(E).T @ f64(E)
    want = np.einsum("xi,ij,xj->x", c, G, c)
    got = oracle.unigram_dist2(W, E)
    assert np.allclose(got, want, rtol=1e-12)
    sel = [7, 0, 149]
    assert np.allclose(oracle.unigram_dist2(W, E, rows=sel), want[sel], rtol=1e-12)


def test_identity_embedding_gives_the_euclidean_distance_from_the_mean():
    V = d = 32
    W = synth.gaussian_weights(V, d, 1.0, 2, "W")
    E = synth.f32_to_bf16_bits(np.eye(V, d, dtype=np.float32))
    c = centred(W)
    assert np.allclose(oracle.unigram_dist2(W, E), (c * c).sum(axis=1), rtol=1e-12)


def test_hand_example():
    # W rows (1,0), (3,0), (2,3): mean (2,1); centred (-1,-1), (1,-1), (0,2).  E rows (1,0), (1,1).
    # d^2 = (c.v_1)^2 + (c.v_2)^2 = 1 + 4, 1 + 0, 0 + 4
    W = synth.f32_to_bf16_bits(np.array([[1, 0], [3, 0], [2, 3]], np.float32))
    E = synth.f32_to_bf16_bits(np.array([[1, 0], [1, 1], [0, 0]], np.float32))
    d2 = oracle.unigram_dist2(W, E)
    assert d2.tolist() == [5.0, 1.0, 4.0]
    assert oracle.smallest_k(d2, 3).tolist() == [1, 2, 0]


def test_shifting_every_output_embedding_changes_nothing():
    g = np.random.default_rng(0)
    Wf = g.integers(-8, 9, (40, 16)).astype(np.float32)          # small integers: exact in bf16, and so is the shift
    E = synth.gaussian_weights(40, 16, 1.0, 3, "E")
    a = oracle.unigram_dist2(synth.f32_to_bf16_bits(Wf), E)
    b = oracle.unigram_dist2(synth.f32_to_bf16_bits(Wf + 4.0), E)
    assert np.allclose(a, b, rtol=1e-12)


def test_smallest_k_orders_ties_by_token_id():
    d2 = np.array([3.0, 1.0, 2.0, 1.0, 0.5, 2.0])
    assert oracle.smallest_k(d2, 5).tolist() == [4, 1, 3, 2, 5]
    assert np.array_equal(oracle.smallest_k(d2, 6), np.argsort(d2, kind="stable"))
