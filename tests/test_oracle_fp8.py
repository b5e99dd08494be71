"""Pins for the oracle's 8-bit (E4M3) head: the format's closed form and published constants, a nearest-value
search written out in numpy, a library cast, and inputs on which quantisation is exact so that the quantised
head must reproduce the bf16 head."""
import numpy as np
import pytest
import torch

import oracle
import synth


def _finite_codes():
    return np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


def test_decode_matches_the_format_definition():
    dec = oracle.e4m3_decode(np.arange(256, dtype=np.uint8))
    # constants of the OCP FP8 E4M3 format: bias 7, largest finite 448, smallest normal 2^-6, smallest subnormal 2^-9
    assert dec[0x38] == 1.0 and dec[0x40] == 2.0 and dec[0x30] == 0.5
    assert dec[0x7E] == 448.0 and dec[0x08] == 2.0 ** -6 and dec[0x01] == 2.0 ** -9 and dec[0x07] == 7 * 2.0 ** -9
    assert np.isnan(dec[0x7F]) and np.isnan(dec[0xFF])
    assert dec[0x00] == 0.0 and dec[0x80] == 0.0 and np.signbit(dec[0x80])
    # closed form, written independently with integer fields
    for c in _finite_codes():
        e, m = (int(c) >> 3) & 15, int(c) & 7
        mag = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
        assert dec[c] == (-mag if c & 0x80 else mag)
    assert np.all(np.diff(dec[:0x7F]) > 0)  # magnitudes ascend with the code
    # library view of the same byte patterns
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    fin = _finite_codes()
    assert np.array_equal(lib[fin], dec[fin])


def _brute_encode(values):
    """Nearest finite magnitude by exhaustive search; ties to the even code; zero keeps no sign."""
    mags = oracle.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    out = np.empty(len(values), dtype=np.uint8)
    for i, v in enumerate(values):
        a = abs(float(v))
        dist = np.abs(mags - a)
        best = np.flatnonzero(dist == dist.min())
        code = int(best[0]) if len(best) == 1 else int([b for b in best if b % 2 == 0][0])
        out[i] = 0 if code == 0 else code | (0x80 if np.signbit(v) else 0)
    return out


def test_encode_is_round_to_nearest_even_with_saturation():
    g = synth.stream(11, "fp8/encode")
    mags = oracle.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    mid = 0.5 * (mags[:-1] + mags[1:])                                   # exact ties
    vals = np.concatenate([
        mags, mid, np.nextafter(mid.astype(np.float32), np.float32(0)), np.nextafter(mid.astype(np.float32), np.float32(1e9)),
        np.exp(g.uniform(np.log(1e-4), np.log(448.0), 4000)), g.uniform(0, 448, 2000), [0.0, 448.0, 1e-12],
    ]).astype(np.float32)
    vals = np.concatenate([vals, -vals])
    got = oracle.e4m3_encode(vals)
    assert np.array_equal(got, _brute_encode(vals))
    # every finite code is a fixed point (except -0, which is stored as +0)
    fin = np.array([c for c in _finite_codes() if c != 0x80], dtype=np.uint8)
    assert np.array_equal(oracle.e4m3_encode(oracle.e4m3_decode(fin).astype(np.float32)), fin)
    # saturation
    assert list(oracle.e4m3_encode(np.array([449, 464, 1e6, 3e38, -449, -1e30], dtype=np.float32))) == [0x7E] * 4 + [0xFE] * 2
    # library cast (round to nearest even) on the unsaturated range; it keeps the sign of zero, this format drops it
    lib = torch.from_numpy(vals).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    lib[(lib & 0x7F) == 0] = 0
    assert np.array_equal(got, lib)


def test_quantize_rows_follows_the_recipe():
    g = synth.stream(12, "fp8/rows")
    X = synth.f32_to_bf16_bits((g.standard_normal((7, 96)) * np.exp(g.uniform(-6, 6, (7, 1)))).astype(np.float32))
    X[3] = 0                                      # an all-zero row
    X[5, 10] = synth.f32_to_bf16_bits(np.array([-0.0], dtype=np.float32))[0]
    codes, scale = oracle.quantize_rows_e4m3(X)
    xf = synth.bf16_bits_to_f32(X)
    for r in range(X.shape[0]):
        amax = np.float32(np.abs(xf[r]).max())
        sc = np.float32(1.0) if amax == 0 else np.float32(amax / np.float32(448.0))
        assert scale[r] == sc
        assert np.array_equal(codes[r], _brute_encode((xf[r] / sc).astype(np.float32)))
    dec = oracle.e4m3_decode(codes)
    assert np.all(np.abs(dec).max(axis=1)[[0, 1, 2, 4, 5, 6]] == 448.0)   # the largest entry maps to the largest code
    assert np.all(codes[3] == 0) and scale[3] == 1.0
    # error bound: half a unit in the last place of a 3-bit mantissa (2^-4 relative) or half the subnormal step
    err = np.abs(dec * scale[:, None].astype(np.float64) - xf)
    bound = np.maximum(np.abs(xf) * 2.0 ** -4, scale[:, None].astype(np.float64) * 2.0 ** -10) * (1 + 1e-6)
    assert np.all(err <= bound)


def test_quantised_head_equals_bf16_head_when_quantisation_is_exact():
    """Rows made of E4M3 values times 2^-8 with 448 * 2^-8 present: scale = 2^-8 and every code is exact."""
    g = synth.stream(13, "fp8/exact")
    V, d, M = 300, 64, 9
    fin = np.array([c for c in _finite_codes() if c != 0x80], dtype=np.uint8)

    def exact_rows(n):
        c = fin[g.integers(0, len(fin), (n, d))]
        c[:, 0] = 0x7E
        return c, synth.f32_to_bf16_bits((oracle.e4m3_decode(c) * 2.0 ** -8).astype(np.float32))

    wc, W = exact_rows(V)
    hc, H = exact_rows(M)
    Wq, ws = oracle.quantize_rows_e4m3(W)
    Hq, hs = oracle.quantize_rows_e4m3(H)
    assert np.array_equal(Wq, wc) and np.array_equal(Hq, hc) and np.all(ws == 2.0 ** -8) and np.all(hs == 2.0 ** -8)
    am8, mx8, gap8 = oracle.verify_q8(Hq, hs, Wq, ws)
    am, mx, gap = oracle.verify(H, W)
    assert np.array_equal(am8, am) and np.allclose(mx8, mx, rtol=1e-13, atol=0) and np.allclose(gap8, gap, rtol=1e-9, atol=1e-12)


def test_quantised_head_against_numpy_matmul():
    g = synth.stream(14, "fp8/matmul")
    V, d, M = 257, 80, 11
    W = synth.f32_to_bf16_bits((g.standard_normal((V, d)) * 0.02).astype(np.float32))
    H = synth.f32_to_bf16_bits(g.standard_normal((M, d)).astype(np.float32))
    Wq, ws = oracle.quantize_rows_e4m3(W)
    Hq, hs = oracle.quantize_rows_e4m3(H)
    z = (oracle.e4m3_decode(Hq) @ oracle.e4m3_decode(Wq).T) * hs[:, None].astype(np.float64) * ws[None, :].astype(np.float64)
    rows = [10, 0, 3]
    am, mx, gap = oracle.verify_q8(Hq, hs, Wq, ws, rows=rows)
    assert np.array_equal(am, z[rows].argmax(axis=1))
    assert np.allclose(mx, z[rows].max(axis=1), rtol=1e-12, atol=1e-15)
    top2 = np.sort(z[rows], axis=1)[:, -2:]
    assert np.allclose(gap, top2[:, 1] - top2[:, 0], rtol=1e-9, atol=1e-12)
    # quantisation error of a logit stays within the bound the per-element error implies
    zb = oracle.logits_rows(H, W)
    xf, wf = np.abs(synth.bf16_bits_to_f32(H).astype(np.float64)), np.abs(synth.bf16_bits_to_f32(W).astype(np.float64))
    assert np.all(np.abs(z - zb) <= (2 * 2.0 ** -4 + 2.0 ** -8) * (xf @ wf.T) + 1e-9)
