"""Memory-safety evidence without a sanitizer: every output lives between guard regions filled with a
sentinel, is itself poison-filled before the call, and every call is run twice and must repeat."""
import numpy as np
import pytest
import torch

import synth
from gpu_util import dev_bf16, dev_i32

pytestmark = pytest.mark.gpu
GUARD = 64          # elements on each side
SENT = -123456789


def guarded(shape, dtype):
    n = int(np.prod(shape))
    byte = dtype == torch.uint8          # E4M3 codes: sentinel 0xA5, poison 0x7F (the NaN code, never produced)
    buf = torch.full((n + 2 * GUARD,), 0xA5 if byte else SENT, dtype=dtype, device="cuda")
    view = buf[GUARD:GUARD + n].view(shape)
    view.fill_(0x7F if byte else -77)    # poison: stale values cannot pass for results
    return buf, view


def intact(buf):
    sent = 0xA5 if buf.dtype == torch.uint8 else SENT
    return bool((buf[:GUARD] == sent).all() and (buf[-GUARD:] == sent).all())


def unwritten(view):
    return bool((view == (0x7F if view.dtype == torch.uint8 else -77)).any())


def test_outputs_stay_inside_their_buffers_and_repeat():
    import paper_2411_03786_b200 as ngs
    V, d, k, w, B, S, cap = 1000, 208, 10, 5, 8, 3, 408
    E = synth.gaussian_weights(V, d, 1.0, 1, "E")
    W = synth.gaussian_weights(V, d, 1.0, 1, "W")
    ctx = ngs.SpecContext(dev_bf16(E), dev_bf16(W))
    lib, h = ngs.load_library(), ctx._h
    import ctypes as C
    P = lambda t: C.c_void_p(t.data_ptr())
    results = []
    for rep in range(2):
        bufs = {}
        def out(name, shape, dtype=torch.int32):
            bufs[name] = guarded(shape, dtype)
            return bufs[name][1]
        tab, val, ext = out("tab", (V, k)), out("val", (V, k), torch.float32), out("ext", (V, k, w))
        assert lib.build_model_ngram_tables(h, None, k, w, P(tab), P(val), P(ext), None) == 0
        uni, d2 = out("uni", (12,)), out("d2", (V,), torch.float32)
        assert lib.build_model_unigram(h, 12, P(uni), P(d2), None) == 0
        hist_h, lens_h, _ = synth.zipf_histories(S, 400, V, 1.1, 0.3, seed=2, cap=cap)
        lens_h[1] = 37
        bufs["hist"] = guarded((S, cap), torch.int32)
        hist = bufs["hist"][1]
        hist.copy_(dev_i32(hist_h))
        lens = dev_i32(lens_h)
        drafts, nd, src, cnt = out("drafts", (S, B, w)), out("nd", (S,)), out("src", (S, B)), out("cnt", (S, B))
        qs = (C.c_int * 2)(2, 1)
        assert lib.draft_context_ngrams(h, P(hist), P(lens), S, cap, qs, 2, 4, B, w, 3, P(drafts), P(nd), P(src), P(cnt), None) == 0
        M = S * B * (w + 1)
        H = dev_bf16(synth.hidden_literal(M, d, seed=3))
        am, mx = out("am", (M,)), out("mx", (M,), torch.float32)
        assert lib.verify_lmhead_argmax(h, P(H), M, P(am), P(mx), None) == 0
        acc, best, com = out("acc", (S,)), out("best", (S,)), out("com", (S, w + 1))
        assert lib.accept_and_commit(h, P(drafts), P(nd), P(am), S, B, w, P(hist), P(lens), cap, P(acc), P(best), P(com), None) == 0
        logits = out("logits", (5, V), torch.float32)
        assert lib.spec_debug_logits(h, P(H), 5, P(logits), None) == 0
        wq, ws = out("wq", (V, d), torch.uint8), out("ws", (V,), torch.float32)
        assert lib.spec_quantize_head_fp8(h, P(wq), P(ws), None) == 0
        hq, hs = out("hq", (M, d), torch.uint8), out("hs", (M,), torch.float32)
        am8, mx8 = out("am8", (M,)), out("mx8", (M,), torch.float32)
        assert lib.verify_lmhead_argmax_fp8(h, P(H), M, P(hq), P(hs), P(am8), P(mx8), None) == 0
        torch.cuda.synchronize()
        assert ctx.get_status() == 0
        for name, (buf, view) in bufs.items():
            assert intact(buf), f"{name}: guard region overwritten"
        for name in ("tab", "val", "ext", "uni", "d2", "nd", "src", "cnt", "am", "mx", "acc", "best", "logits", "wq", "ws", "hq", "hs",
                     "am8", "mx8"):
            assert not unwritten(bufs[name][1]), f"{name}: element left unwritten"
        results.append({n: v.clone() for n, (b, v) in bufs.items()})
    for name in results[0]:
        assert torch.equal(results[0][name], results[1][name]), f"{name}: two identical calls disagree"
    ctx.close()
