"""GPU parity of the 8-bit (E4M3) verification head: the quantiser byte for byte, the head against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import dev_bf16, weights

pytestmark = pytest.mark.gpu
TOL = 2e-2   # logit tolerance: products of E4M3 values are exact, fp32 accumulation of d terms is far inside it


@pytest.fixture(scope="module")
def ngs():
    import paper_2411_03786_b200 as m
    return m


def rows_with_spread(n, d, seed):
    """Gaussian rows with row scales over several decades, an all-zero row, signed zeros and tiny entries."""
    g = synth.stream(seed, "fp8/gpu-rows")
    x = (g.standard_normal((n, d)) * np.exp(g.uniform(-8, 8, (n, 1)))).astype(np.float32)
    x[g.random((n, d)) < 0.02] *= 1e-4         # entries that land in the subnormal range or round to zero
    bits = synth.f32_to_bf16_bits(x)
    if n > 2:
        bits[1] = 0
        bits[2, ::3] = 0x8000                  # -0.0
    return bits


@pytest.mark.parametrize("n,d", [(1, 16), (5, 80), (37, 128), (300, 4096), (64, 272)])
def test_quantiser_is_bit_exact(ngs, n, d):
    W = synth.gaussian_weights(64, d, 1.0, 3, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    X = rows_with_spread(n, d, seed=n + d)
    codes, scale = ctx.quantize_rows_fp8(dev_bf16(X))
    ref_codes, ref_scale = oracle.quantize_rows_e4m3(X)
    assert np.array_equal(scale.cpu().numpy().view(np.uint32), ref_scale.view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), ref_codes)
    assert ctx.get_status() == 0
    ctx.close()


# one tile, ragged V / K tails (d % 128 != 0), two m-tiles in one pass, several m-tiles
SHAPES = [(1024, 128, 20), (1000, 208, 150), (4136, 320, 300), (96, 64, 1), (33, 16, 129), (4136, 320, 256), (9000, 144, 200),
          (5000, 4096, 200), (2100, 2048, 130),                      # two m-tiles in one pass, k-loop longer than the ring
          (40000, 256, 200), (40000, 2048, 140), (40000, 512, 60)]    # ... and more than one 256-column tile per CTA


@pytest.mark.parametrize("V,d,M", SHAPES)
def test_fp8_verify_matches_oracle(ngs, V, d, M):
    W = synth.gaussian_weights(V, d, d ** -0.5, V + d + 2, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    wq, ws = ctx.quantize_head_fp8()
    Wq, Ws = oracle.quantize_rows_e4m3(W)
    assert np.array_equal(wq.cpu().numpy(), Wq) and np.array_equal(ws.cpu().numpy(), Ws)
    H = synth.hidden_literal(M, d, seed=M + 2)
    Hq, Hs = oracle.quantize_rows_e4m3(H)
    ref_am, ref_mx, gap = oracle.verify_q8(Hq, Hs, Wq, Ws)
    for rep in range(2):      # the second call checks that the merge scratch was re-armed
        am, mx = ctx.verify_lmhead_argmax_fp8(dev_bf16(H), with_max=True)
        am, mx = am.cpu().numpy(), mx.cpu().numpy().astype(np.float64)
        bad = am != ref_am
        assert not (bad & (gap >= TOL)).any(), f"{bad.sum()} mismatches with clear margins"
        assert np.abs(mx - ref_mx).max() <= TOL
    # hidden states quantised by the caller beforehand
    scratch = ctx.quantize_rows_fp8(dev_bf16(H))
    am2, _ = ctx.verify_lmhead_argmax_fp8(None, scratch=scratch)
    assert np.array_equal(am2.cpu().numpy(), am)
    assert ctx.get_status() == 0
    ctx.close()


def test_fp8_exact_ties_take_the_lowest_token(ngs):
    V, d = 700, 128
    W = synth.gaussian_weights(V, d, 1.0, 9, "W")
    W[[40, 300, 650]] = W[5]
    W[[6, 9, 17, 31]] = W[5]               # ties inside one 32-column chunk, at every level of its comparison tree
    W[[101, 99, 110]] = W[98]
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    ctx.quantize_head_fp8()
    am, _ = ctx.verify_lmhead_argmax_fp8(dev_bf16(W[[5, 650, 110, 31]].copy()))
    assert am.cpu().tolist() == [5, 5, 98, 5]
    ctx.close()


def test_fp8_needs_a_head_first(ngs):
    W = synth.gaussian_weights(64, 64, 1.0, 1, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    with pytest.raises(ngs.SpecError, match="spec_quantize_head_fp8"):
        ctx.verify_lmhead_argmax_fp8(dev_bf16(W[:4].copy()))
    ctx.close()
    W8 = synth.gaussian_weights(64, 72, 1.0, 1, "W")     # d % 16 != 0
    ctx = ngs.SpecContext(dev_bf16(W8), dev_bf16(W8))
    with pytest.raises(ngs.SpecError, match="16"):
        ctx.quantize_head_fp8()
    ctx.close()


def test_fp8_verify_full_size_C2(ngs):
    """The benchmark's launch configuration: V=32000, d=4096, M=48, planted targets and literal noise."""
    c = synth.config("C2")
    W = weights(c, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    wq, ws = ctx.quantize_head_fp8()
    Wq, Ws = oracle.quantize_rows_e4m3(W)
    assert np.array_equal(wq.cpu().numpy(), Wq) and np.array_equal(ws.cpu().numpy(), Ws)
    g = synth.stream(c["seed"], "fp8/targets")
    targets = g.integers(0, c["V"], c["M"]).astype(np.int32)
    for H, planted in ((synth.hidden_planted(W, targets, seed=c["seed"]), True), (synth.hidden_literal(c["M"], c["d"], seed=5), False)):
        Hq, Hs = oracle.quantize_rows_e4m3(H)
        ref_am, ref_mx, gap = oracle.verify_q8(Hq, Hs, Wq, Ws)
        am, mx = ctx.verify_lmhead_argmax_fp8(dev_bf16(H), with_max=True)
        am, mx = am.cpu().numpy(), mx.cpu().numpy().astype(np.float64)
        bad = am != ref_am
        assert not (bad & (gap >= TOL)).any()
        assert np.abs(mx - ref_mx).max() <= TOL
        if planted:   # the planted margin (about 14) dwarfs the quantisation error: 8-bit and bf16 heads agree
            assert np.array_equal(am, targets)
            am16, _ = ctx.verify_lmhead_argmax(dev_bf16(H))
            assert np.array_equal(am16.cpu().numpy(), am)
    assert ctx.get_status() == 0
    ctx.close()


@pytest.mark.parametrize("name", ["C3", "C4"])
def test_fp8_verify_full_size_sampled_rows(ngs, name):
    """Tensor-bound launch shapes of the benchmark (several m-tiles, V=32000 and V=128256): all M rows on the GPU,
    a seeded sample of rows (tile edges included) through the oracle."""
    c = synth.config(name)
    W = weights(c, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    wq, ws = ctx.quantize_head_fp8()
    Wq, Ws = oracle.quantize_rows_e4m3(W)
    assert np.array_equal(ws.cpu().numpy(), Ws)
    g = synth.stream(c["seed"], "fp8/rows-checked")
    M = c["M"]
    rows = np.array(sorted({0, 1, 127, 128, M - 1, M - 2, (M - 1) // 128 * 128} | set(g.integers(0, M, 9).tolist())), dtype=np.int64)
    assert np.array_equal(wq.cpu().numpy()[rows % c["V"]], Wq[rows % c["V"]])
    H = synth.hidden_literal(M, c["d"], seed=c["seed"] + 8)
    targets = g.integers(0, c["V"], M).astype(np.int32)
    H[::2] = synth.hidden_planted(W, targets[::2], seed=c["seed"] + 9)      # every other row has a planted arg max
    am, mx = ctx.verify_lmhead_argmax_fp8(dev_bf16(H), with_max=True)
    am, mx = am.cpu().numpy(), mx.cpu().numpy().astype(np.float64)
    Hq, Hs = oracle.quantize_rows_e4m3(H[rows])
    ref_am, ref_mx, gap = oracle.verify_q8(Hq, Hs, Wq, Ws)
    bad = am[rows] != ref_am
    assert not (bad & (gap >= TOL)).any()
    assert np.abs(mx[rows] - ref_mx).max() <= TOL
    assert np.array_equal(am[::2], targets[::2])
    assert am.min() >= 0 and am.max() < c["V"]
    assert ctx.get_status() == 0
    ctx.close()
