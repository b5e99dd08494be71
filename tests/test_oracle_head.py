"""Pins for the oracle's LM-head routines (model bigram table, verification argmax)."""
import numpy as np
import torch

import oracle
import synth


def f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def test_bf16_rounding_matches_a_library_conversion():
    x = synth.stream(5, "r").standard_normal(10000, dtype=np.float32) * 3
    x[:6] = np.array([1.00390625, 1.01171875, -1.00390625, 65504.0, 1e-40, -0.0], dtype=np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.round_to_bf16(x), ref)


def test_logits_against_library_matmul():
    A = synth.gaussian_weights(37, 96, 1.0, 1, "A")
    W = synth.gaussian_weights(203, 96, 1.0, 1, "W")
    z = oracle.logits_rows(A, W)
    ref = f64(A) @ f64(W).T
    assert z.shape == (37, 203) and np.abs(z - ref).max() < 1e-12
    sel = [5, 0, 36, 5]
    assert np.abs(oracle.logits_rows(A, W, rows=sel) - ref[sel]).max() < 1e-12
    # a transposed or swapped operand would fail this asymmetric check
    assert abs(z[3, 100] - float(f64(A)[3] @ f64(W)[100])) < 1e-12


def test_table_against_full_sort_on_tiny_config():
    c = synth.config("C1")
    E = synth.f32_to_bf16_bits(synth.gaussian_weights(c["V"], c["d"], c["wstd"], 0, "E", "f32"))
    W = synth.f32_to_bf16_bits(synth.gaussian_weights(c["V"], c["d"], c["wstd"], 0, "W", "f32"))
    idx, val = oracle.model_table(E, W, 4)
    z = f64(E) @ f64(W).T
    order = np.argsort(-z, axis=1, kind="stable")[:, :4]     # stable: equal values keep ascending id
    assert np.array_equal(idx, order.astype(np.int32))
    assert np.abs(val - np.take_along_axis(z, order, 1)).max() < 1e-12
    am, mx, gap = oracle.verify(E, W)
    assert np.array_equal(am, order[:, 0]) and np.abs(mx - val[:, 0]).max() < 1e-12
    assert np.abs(gap - (val[:, 0] - val[:, 1])).max() < 1e-12 and (gap >= 0).all()


def test_tied_unit_norm_weights_predict_the_token_itself():
    # Cauchy-Schwarz: for distinct unit rows <u_x, u_y> < 1 = <u_x, u_x>.  bf16 rounding
    # perturbs norms by < 2^-8, far less than the gap between random directions.
    U = synth.unit_rows_bf16(synth.gaussian_weights(300, 64, 1.0, 2, "U", "f32"))
    idx, _ = oracle.model_table(U, U, 3)
    assert np.array_equal(idx[:, 0], np.arange(300))
    am, _, _ = oracle.verify(U, U)
    assert np.array_equal(am, np.arange(300))


def test_permutation_weights_give_the_planted_bigram_and_chain():
    V = d = 48
    g = np.random.default_rng(0)
    pi = g.permutation(V)
    A = synth.f32_to_bf16_bits(np.eye(V, d, dtype=np.float32))
    Wf = np.zeros((V, d), dtype=np.float32)
    Wf[pi, np.arange(V)] = 1.0                    # row pi(x) of W is e_x  =>  <A[x], W[pi(x)]> = 1
    Wf[(pi + 1) % V, np.arange(V)] += 0.5         # runner-up at pi(x)+1
    W = synth.f32_to_bf16_bits(Wf)
    idx, val = oracle.model_table(A, W, 2)
    assert np.array_equal(idx[:, 0], pi) and np.array_equal(idx[:, 1], (pi + 1) % V)
    assert np.allclose(val, [[1.0, 0.5]] * V)
    ext = oracle.extend_table(idx, 4)
    for x in (0, 7, 47):
        chain, s = [], pi[x]
        for _ in range(4):
            chain.append(s)
            s = pi[s]
        assert ext[x, 0].tolist() == chain
        chain2, s = [], (pi[x] + 1) % V
        for _ in range(4):
            chain2.append(s)
            s = pi[s]
        assert ext[x, 1].tolist() == chain2


def test_exact_ties_go_to_the_lower_token_id():
    W = synth.gaussian_weights(40, 32, 1.0, 3, "W")
    W[[5, 17, 30]] = W[11]                         # four identical rows: 5, 11, 17, 30
    A = W[[11]].copy()                             # its own direction wins
    idx, val = oracle.model_table(A, W, 6)
    assert idx[0, :4].tolist() == [5, 11, 17, 30] and len(set(val[0, :4])) == 1
    am, _, gap = oracle.verify(A, W)
    assert am[0] == 5 and gap[0] == 0.0
