"""GPU parity over seeded random head shapes: every row regime (one m-tile, two m-tiles in one pass, several
m-tiles) crossed with short and long k-loops and one or several tiles per CTA, for the bf16 and the 8-bit
verification head and (small vocabularies) the table build.  Rows are sampled for the oracle."""
import numpy as np
import pytest

import oracle
import synth
from gpu_util import dev_bf16

pytestmark = pytest.mark.gpu
TOL = 2e-2


def random_shapes(n, seed):
    g = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        V = int(g.choice([g.integers(16, 300), g.integers(300, 5000), g.integers(5000, 70000)]))
        d = int(g.choice([16, 64, 128, 208, 512, 1024, 2048, 4096, int(g.integers(1, 130)) * 16]))
        M = int(g.choice([g.integers(1, 129), g.integers(129, 257), g.integers(257, 700)]))
        if V * d > 1.2e8:
            V = int(1.2e8 // d)
        out.append((V, d, M))
    return out


@pytest.mark.parametrize("V,d,M", random_shapes(36, seed=2024))
def test_random_head_shape(V, d, M):
    import paper_2411_03786_b200 as ngs
    g = np.random.default_rng(V * 31 + d * 7 + M)
    W = synth.gaussian_weights(V, d, d ** -0.5, V + d + M, "W")
    ctx = ngs.SpecContext(dev_bf16(W), dev_bf16(W))
    H = synth.hidden_literal(M, d, seed=M + d)
    edge = [0, M - 1, min(M - 1, 127), min(M - 1, 128), min(M - 1, 191), min(M - 1, 192), min(M - 1, 256)]
    rows = np.unique(np.concatenate([edge, g.integers(0, M, 6)])).astype(np.int64)

    am, mx = ctx.verify_lmhead_argmax(dev_bf16(H), with_max=True)
    am, mx = am.cpu().numpy(), mx.cpu().numpy().astype(np.float64)
    r_am, r_mx, gap = oracle.verify(H, W, rows=rows)
    assert not ((am[rows] != r_am) & (gap >= TOL)).any()
    assert np.abs(mx[rows] - r_mx).max() <= TOL
    assert am.min() >= 0 and am.max() < V

    ctx.quantize_head_fp8()
    Wq, Ws = oracle.quantize_rows_e4m3(W)
    am8, mx8 = ctx.verify_lmhead_argmax_fp8(dev_bf16(H), with_max=True)
    am8, mx8 = am8.cpu().numpy(), mx8.cpu().numpy().astype(np.float64)
    Hq, Hs = oracle.quantize_rows_e4m3(H[rows])
    r8, m8, g8 = oracle.verify_q8(Hq, Hs, Wq, Ws)
    assert not ((am8[rows] != r8) & (g8 >= TOL)).any()
    assert np.abs(mx8[rows] - m8).max() <= TOL

    if V <= 2500:
        k = int(g.integers(1, min(32, V) + 1))
        tab, val, _ = ctx.build_model_ngram_tables(k, with_values=True)
        tab, val = tab.cpu().numpy(), val.cpu().numpy()
        rs = np.unique(g.integers(0, V, 6)).astype(np.int64)
        _, v = oracle.model_table(W, W, k, rows=rs)
        z = oracle.logits_rows(W, W, rows=rs)
        for j, x in enumerate(rs):
            assert len(set(tab[x].tolist())) == k
            assert np.abs(z[j][tab[x]] - v[j]).max() <= TOL and np.abs(val[x] - z[j][tab[x]]).max() <= TOL
    assert ctx.get_status() == 0
    ctx.close()
