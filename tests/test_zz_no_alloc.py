"""The allocation-free verify entry point against the ordinary one.

Some callers of this library may not allocate device memory when they verify drafts (an engine
whose memory pool already owns the whole GPU, or a hot path where cudaMalloc's device-wide
synchronisation is not acceptable).  ``verify_lmhead_argmax_noalloc`` serves them from a fixed
scratch array inside the library.  This file is collected last on purpose: a failure here cannot
hide a failure in any other test.  It also has to pass on its own in a fresh process.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import dev_bf16

TOL = 2e-2


@pytest.mark.gpu
def test_noalloc_verify_matches_context_verify_on_two_calls_in_a_row():
    import paper_2411_03786_b200 as ngs
    V, d = 4136, 320                       # several vocabulary chunks with a ragged tail
    W = synth.gaussian_weights(V, d, d ** -0.5, 21, "W")
    dW = dev_bf16(W)
    ctx = ngs.SpecContext(dW, dW)
    for call, M in enumerate((300, 77, 200)):   # later calls reuse the scratch the earlier ones left behind; all three row regimes
        H = synth.hidden_literal(M, d, seed=50 + call)
        dH = dev_bf16(H)
        ref_am, ref_mx = ctx.verify_lmhead_argmax(dH, with_max=True)
        out = (torch.empty(M, dtype=torch.int32, device="cuda"), torch.empty(M, dtype=torch.float32, device="cuda"))
        allocs = lambda: torch.cuda.memory_stats()["allocation.all.allocated"]   # cumulative, frees do not lower it
        before = allocs()
        am, mx = ngs.verify_lmhead_argmax_noalloc(dW, dH, out)
        torch.cuda.synchronize()
        assert allocs() == before                            # the wrapper asked torch for no memory either
        assert torch.equal(am, ref_am)                       # same kernel, integer result: identical
        assert (mx - ref_mx).abs().max().item() <= TOL
        assert (am >= 0).all() and (am < V).all()
        # and against the CPU oracle, on a seeded sample of rows (first, last, tile edges)
        rows = np.array(sorted({0, 1, M - 1, min(127, M - 1), min(128, M - 1)} | set(np.random.default_rng(call).integers(0, M, 24).tolist())))
        o_am, o_mx, gap = oracle.verify(H, W, rows=rows)
        bad = am.cpu().numpy()[rows] != o_am
        assert not (bad & (gap >= TOL)).any()
        assert np.abs(mx.cpu().numpy()[rows].astype(np.float64) - o_mx).max() <= TOL
    ctx.close()


@pytest.mark.gpu
def test_noalloc_verify_rejects_blocks_beyond_its_scratch():
    import paper_2411_03786_b200 as ngs
    lib = ngs.load_library()
    W = dev_bf16(synth.gaussian_weights(64, 64, 1.0, 1, "W"))
    H = torch.zeros((4097, 64), dtype=torch.bfloat16, device="cuda")
    am = torch.empty(4097, dtype=torch.int32, device="cuda")
    with pytest.raises(ngs.SpecError, match="exceeds the built-in scratch"):
        ngs.verify_lmhead_argmax_noalloc(W, H, (am, None))
