"""CPU oracle for the batched N-gram speculation step (arXiv 2411.03786).

TEST INFRASTRUCTURE ONLY.  This package wraps ``ngram_oracle.c`` (plain C, fp64)
with ctypes and adds the toy-model decode loops.  It is independent of the CUDA
library: neither imports the other and they share no code.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may call it.

bf16 matrices are ``numpy.uint16`` bit patterns; token arrays are ``int32``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ngram_oracle.c")
_LIB = os.path.join(_HERE, "libngram_oracle.so")
_lib = None

FLAG_DEDUP = 1
FLAG_MODEL_FILL = 2
FLAG_KEY_NEXT_TOKEN = 4
FLAG_PARTIAL_TAIL = 8


def flag_reserve(n: int) -> int:
    """Flag bits that reserve ``n`` draft rows for the model strategy."""
    return (int(n) & 0xFF) << 8


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over independent rows / sequences)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c99", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_f32_to_bf16.restype = C.c_uint16
        _lib.oracle_f32_to_bf16.argtypes = [C.c_float]
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 matrices are passed as uint16 bit patterns"
    return a


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bits, round-to-nearest-even (the one rounding fp32 weights get)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_round_to_bf16(_p(x, C.c_float), _p(out, C.c_uint16), C.c_long(x.size))
    return out


def context_draft(hist, q: int, w: int, topk: int, key_len: int | None = None):
    """Section 4.2: top continuations after earlier occurrences of the last q tokens.

    ``key_len`` (default w) = how many continuation tokens identify a group.
    Returns ``(rows[n, w], counts[n], last_start[n])`` with n <= topk.
    """
    hist = _i32(hist)
    rows = np.full((max(topk, 1), w), -1, dtype=np.int32)
    counts = np.zeros(max(topk, 1), dtype=np.int32)
    lasts = np.zeros(max(topk, 1), dtype=np.int32)
    n = lib().oracle_context_draft_keyed(_p(hist, C.c_int32), int(hist.size), int(q), int(w),
                                         int(w if key_len is None else key_len), int(topk),
                                         _p(rows, C.c_int32), _p(counts, C.c_int32), _p(lasts, C.c_int32))
    return rows[:n].copy(), counts[:n].copy(), lasts[:n].copy()


def context_draft_partial(hist, q: int, w: int, topk: int, key_len: int | None = None):
    """The variant in which occurrences with fewer than w following tokens count too, their continuation
    extended periodically.  Returns ``(rows[n, w], counts[n], last_start[n])`` with n <= topk."""
    hist = _i32(hist)
    rows = np.full((max(topk, 1), w), -1, dtype=np.int32)
    counts = np.zeros(max(topk, 1), dtype=np.int32)
    lasts = np.zeros(max(topk, 1), dtype=np.int32)
    n = lib().oracle_context_draft_partial(_p(hist, C.c_int32), int(hist.size), int(q), int(w),
                                           int(w if key_len is None else key_len), int(topk),
                                           _p(rows, C.c_int32), _p(counts, C.c_int32), _p(lasts, C.c_int32))
    return rows[:n].copy(), counts[:n].copy(), lasts[:n].copy()


def extend_table(T, w: int) -> np.ndarray:
    """Section 4.1 "Extensions": ext[x, r, :] = rank-r bigram token then top-1 chaining."""
    T = _i32(T)
    V, k = T.shape
    ext = np.empty((V, k, w), dtype=np.int32)
    lib().oracle_extend_table(_p(T, C.c_int32), V, k, int(w), _p(ext, C.c_int32))
    return ext


def draft_batch(hist, lens, qs, topk: int, B: int, w: int, flags: int = FLAG_DEDUP | FLAG_MODEL_FILL, T=None, V: int | None = None):
    """Section 4.3 mixed strategy for S sequences.  Returns drafts[S,B,w], n_drafts[S], src[S,B], counts[S,B].

    ``V`` (default: the table's row count, else unknown) is the vocabulary size: when known, a context
    row holding a token outside [0, V) is passed over."""
    hist = _i32(hist)
    lens = _i32(lens)
    S, cap = hist.shape
    qs_arr = (C.c_int * max(1, len(qs)))(*[int(q) for q in qs])
    drafts = np.empty((S, B, w), dtype=np.int32)
    nd = np.empty(S, dtype=np.int32)
    src = np.empty((S, B), dtype=np.int32)
    counts = np.empty((S, B), dtype=np.int32)
    if T is not None:
        T = _i32(T)
        k_tab = T.shape[1]
        V = T.shape[0] if V is None else V
    else:
        V, k_tab = (0 if V is None else V), 0
    lib().oracle_draft_batch(_p(hist, C.c_int32), _p(lens, C.c_int32), S, cap, qs_arr, len(qs), int(topk), int(B),
                             int(w), int(flags), _p(T, C.c_int32), V, k_tab,
                             _p(drafts, C.c_int32), _p(nd, C.c_int32), _p(src, C.c_int32), _p(counts, C.c_int32))
    return drafts, nd, src, counts


def _rowsel(rows, n_total):
    if rows is None:
        return None, n_total
    r = np.ascontiguousarray(rows, dtype=np.int64)
    return r, int(r.size)


def logits_rows(A, W, rows=None) -> np.ndarray:
    """fp64 logits ``A[rows] @ W.T`` over bf16 inputs."""
    A, W = _u16(A), _u16(W)
    V, d = W.shape
    r, n = _rowsel(rows, A.shape[0])
    out = np.empty((n, V), dtype=np.float64)
    lib().oracle_logits_rows(_p(A, C.c_uint16), _p(r, C.c_int64), n, _p(W, C.c_uint16), V, d, _p(out, C.c_double))
    return out


def model_table(A, W, k_tab: int, rows=None):
    """Section 4.1 "Bigram": per row the k_tab largest head logits (value desc, id asc)."""
    A, W = _u16(A), _u16(W)
    V, d = W.shape
    r, n = _rowsel(rows, A.shape[0])
    idx = np.empty((n, k_tab), dtype=np.int32)
    val = np.empty((n, k_tab), dtype=np.float64)
    lib().oracle_topk_rows(_p(A, C.c_uint16), _p(r, C.c_int64), n, _p(W, C.c_uint16), V, d, int(k_tab),
                           _p(idx, C.c_int32), _p(val, C.c_double))
    return idx, val


def verify(H, W, rows=None):
    """Greedy next token per position: ``(argmax[n], max[n], top-2 gap[n])``."""
    H, W = _u16(H), _u16(W)
    V, d = W.shape
    r, n = _rowsel(rows, H.shape[0])
    am = np.empty(n, dtype=np.int32)
    mx = np.empty(n, dtype=np.float64)
    gap = np.empty(n, dtype=np.float64)
    lib().oracle_verify_rows(_p(H, C.c_uint16), _p(r, C.c_int64), n, _p(W, C.c_uint16), V, d,
                             _p(am, C.c_int32), _p(mx, C.c_double), _p(gap, C.c_double))
    return am, mx, gap


def e4m3_decode(codes) -> np.ndarray:
    """Value of each OCP E4M3 code (fp64; 0x7F and 0xFF are NaN)."""
    lib().oracle_e4m3_decode.restype = C.c_double
    lib().oracle_e4m3_decode.argtypes = [C.c_uint8]
    codes = np.asarray(codes, dtype=np.uint8)
    return np.array([lib().oracle_e4m3_decode(int(c)) for c in codes.reshape(-1)], dtype=np.float64).reshape(codes.shape)


def e4m3_encode(values) -> np.ndarray:
    """Nearest E4M3 code of each fp32 value (ties to even, saturating at 448, zero stored as +0)."""
    lib().oracle_e4m3_encode.restype = C.c_uint8
    lib().oracle_e4m3_encode.argtypes = [C.c_float]
    values = np.asarray(values, dtype=np.float32)
    return np.array([lib().oracle_e4m3_encode(float(v)) for v in values.reshape(-1)], dtype=np.uint8).reshape(values.shape)


def quantize_rows_e4m3(X):
    """Per-row 8-bit quantisation of a bf16 matrix: ``(codes[R, d] uint8, scale[R] float32)``."""
    X = _u16(X)
    R, d = X.shape
    codes = np.empty((R, d), dtype=np.uint8)
    scale = np.empty(R, dtype=np.float32)
    lib().oracle_quantize_rows_e4m3(_p(X, C.c_uint16), C.c_long(R), d, _p(codes, C.c_uint8), _p(scale, C.c_float))
    return codes, scale


def verify_q8(Hq, hscale, Wq, wscale, rows=None):
    """Greedy next token over the quantised head: ``(argmax[n], max[n], top-2 gap[n])``."""
    Hq, Wq = np.ascontiguousarray(Hq, dtype=np.uint8), np.ascontiguousarray(Wq, dtype=np.uint8)
    hscale = np.ascontiguousarray(hscale, dtype=np.float32)
    wscale = np.ascontiguousarray(wscale, dtype=np.float32)
    V, d = Wq.shape
    r, n = _rowsel(rows, Hq.shape[0])
    am = np.empty(n, dtype=np.int32)
    mx = np.empty(n, dtype=np.float64)
    gap = np.empty(n, dtype=np.float64)
    lib().oracle_verify_rows_q8(_p(Hq, C.c_uint8), _p(hscale, C.c_float), _p(r, C.c_int64), n, _p(Wq, C.c_uint8),
                                _p(wscale, C.c_float), V, d, _p(am, C.c_int32), _p(mx, C.c_double), _p(gap, C.c_double))
    return am, mx, gap


def unigram_dist2(W, E, rows=None) -> np.ndarray:
    """Section 4.1 "Unigram": squared distance of each output embedding from the mean, in the metric
    induced by the input embeddings (centred rows rounded to bf16, the rest fp64)."""
    W, E = _u16(W), _u16(E)
    V, d = W.shape
    r, n = _rowsel(rows, V)
    out = np.empty(n, dtype=np.float64)
    lib().oracle_unigram_dist2(_p(W, C.c_uint16), _p(E, C.c_uint16), V, d, _p(r, C.c_int64), n, _p(out, C.c_double))
    return out


def smallest_k(dist2, k: int) -> np.ndarray:
    """Top-k unigram tokens: smallest distance first, equal distances by ascending id."""
    dist2 = np.ascontiguousarray(dist2, dtype=np.float64)
    idx = np.empty(k, dtype=np.int32)
    lib().oracle_smallest_k(_p(dist2, C.c_double), int(dist2.size), int(k), _p(idx, C.c_int32))
    return idx


def accept_commit(drafts, n_drafts, P, hist, lens):
    """Greedy acceptance + commit.  ``hist`` and ``lens`` are updated in place.

    Returns ``(acc_len[S], best_row[S], committed[S, w+1])``.
    """
    drafts, n_drafts, P = _i32(drafts), _i32(n_drafts), _i32(P)
    assert hist.dtype == np.int32 and lens.dtype == np.int32 and hist.flags.c_contiguous
    S, B, w = drafts.shape
    cap = hist.shape[1]
    acc = np.empty(S, dtype=np.int32)
    best = np.empty(S, dtype=np.int32)
    com = np.empty((S, w + 1), dtype=np.int32)
    lib().oracle_accept_commit(_p(drafts, C.c_int32), _p(n_drafts, C.c_int32), _p(P, C.c_int32), S, B, w,
                               _p(hist, C.c_int32), _p(lens, C.c_int32), cap,
                               _p(acc, C.c_int32), _p(best, C.c_int32), _p(com, C.c_int32))
    return acc, best, com


def accumulate_stats(acc_len, best_row, src, w: int, stats=None) -> np.ndarray:
    """Section 5.2 ablation counters: ``[w+1]`` accepted lengths, ``[B]`` accepted row index, ``[5]`` strategy of
    the accepted row, ``[5]`` rows allocated per strategy (index = q, 0 = model); int64, accumulated."""
    acc_len, best_row, src = _i32(acc_len), _i32(best_row), _i32(src)
    S, B = src.shape
    if stats is None:
        stats = np.zeros((w + 1) + B + 10, dtype=np.int64)
    lib().oracle_accumulate_stats(_p(acc_len, C.c_int32), _p(best_row, C.c_int32), _p(src, C.c_int32), S, B, int(w),
                                  _p(stats, C.c_longlong))
    return stats


# ----------------------------------------------------------------------------- toy-model decode loops
def toy_greedy(x0: int, n: int, Hall, W) -> list[int]:
    """Plain greedy decoding: x_{t+1} = argmax_y <Hall[x_t], W[y]>, one token per call."""
    out, x = [], int(x0)
    for _ in range(n):
        am, _, _ = verify(Hall, W, rows=[x])
        x = int(am[0])
        out.append(x)
    return out


def toy_speculative(prompt, n: int, Hall, W, T, qs, topk: int, B: int, w: int,
                    flags: int = FLAG_DEDUP | FLAG_MODEL_FILL, drafts_override=None):
    """Guess-and-verify decoding on the toy model whose hidden state after token x is Hall[x].

    Each step: draft (Section 4.3) -> verify block rows [x_L, s_1..s_w] -> greedy
    acceptance.  Returns ``(generated tokens, per-step accepted lengths, per-step best rows)``.
    ``drafts_override(step, hist, L) -> (drafts[1,B,w], n_drafts[1])`` substitutes arbitrary drafts.
    """
    prompt = list(int(t) for t in prompt)
    cap = (len(prompt) + n + w + 1 + 3) // 4 * 4
    hist = np.full((1, cap), -1, dtype=np.int32)
    hist[0, :len(prompt)] = prompt
    lens = np.array([len(prompt)], dtype=np.int32)
    accs, bests, step = [], [], 0
    while lens[0] - len(prompt) < n:
        L = int(lens[0])
        if drafts_override is not None:
            drafts, nd = drafts_override(step, hist, L)
        else:
            drafts, nd, _, _ = draft_batch(hist, lens, qs, topk, B, w, flags, T)
        block = np.empty((B, w + 1), dtype=np.int64)
        block[:, 0] = hist[0, L - 1]
        block[:, 1:] = np.where(drafts[0] >= 0, drafts[0], 0)
        am, _, _ = verify(Hall, W, rows=block.reshape(-1))
        P = am.reshape(1, B, w + 1)
        acc, best, _ = accept_commit(drafts, nd, P, hist, lens)
        accs.append(int(acc[0]))
        bests.append(int(best[0]))
        step += 1
    gen = hist[0, len(prompt):len(prompt) + n].tolist()
    return gen, accs, bests
