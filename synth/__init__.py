"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This module only draws random numbers and lays them out as arrays.  It holds none
of the speculation method's arithmetic (no matching, counting, top-k, contraction,
argmax or acceptance): those live, separately, in ``oracle/`` and in the CUDA
library.  Both sides read the arrays produced here, so a parity failure can never
be blamed on two generators disagreeing.

bfloat16 arrays are carried as ``numpy.uint16`` bit patterns (numpy has no bf16).
Random streams come from numpy's counter-based Philox generator keyed by
``(seed, stream name)``, so every array is reproducible on its own.
"""
from __future__ import annotations

import hashlib

import numpy as np

__all__ = [
    "stream", "f32_to_bf16_bits", "bf16_bits_to_f32", "gaussian_weights", "zipf_cdf",
    "zipf_histories", "hidden_literal", "hidden_planted", "planted_targets",
    "unit_rows_bf16", "CONFIGS", "config",
]


def stream(seed: int, name: str) -> np.random.Generator:
    """Independent Philox stream for ``(seed, name)``."""
    h = hashlib.sha256(f"{seed}:{name}".encode()).digest()
    key = np.frombuffer(h[:16], dtype=np.uint64).copy()
    return np.random.Generator(np.random.Philox(key=key))


# ----------------------------------------------------------------------------- bf16 storage
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even), returned as uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def gaussian_weights(V: int, d: int, std: float, seed: int, name: str, dtype: str = "bf16") -> np.ndarray:
    """``[V, d]`` matrix ~ N(0, std^2).  dtype "f32" -> float32, "bf16" -> uint16 bits."""
    g = stream(seed, name)
    w = g.standard_normal((V, d), dtype=np.float32) * np.float32(std)
    return w if dtype == "f32" else f32_to_bf16_bits(w)


def unit_rows_bf16(E: np.ndarray) -> np.ndarray:
    """Rows of ``E`` scaled to unit Euclidean length, stored as bf16 bits.

    This is the toy model's hidden-state matrix: row x is what the toy model feeds
    to the LM head after reading token x.
    """
    e = E.astype(np.float64) if E.dtype != np.uint16 else bf16_bits_to_f32(E).astype(np.float64)
    n = np.sqrt((e * e).sum(axis=1, keepdims=True))
    n[n == 0] = 1.0
    return f32_to_bf16_bits((e / n).astype(np.float32))


# ----------------------------------------------------------------------------- token histories
def zipf_cdf(V: int, s: float) -> np.ndarray:
    p = np.arange(1, V + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(p)
    return c / c[-1]


def _zipf_tokens(g: np.random.Generator, n: int, cdf: np.ndarray, perm: np.ndarray) -> np.ndarray:
    r = np.searchsorted(cdf, g.random(n), side="left")
    return perm[np.minimum(r, len(cdf) - 1)].astype(np.int32)


def zipf_histories(S: int, L: int, V: int, s: float, copy_frac: float, seed: int,
                   cap: int | None = None, span=(8, 24), name: str = "hist"):
    """``S`` token histories of length ``L`` with repeated spans.

    Left to right, each event is either one fresh token (finite Zipf(s) over the
    vocabulary, ranks mapped to ids by a seeded permutation) or, with probability
    pi = f / (f + m (1 - f)) (m = mean span length, f = ``copy_frac``), a span of
    uniform length in ``span`` copied token by token from a uniformly chosen earlier
    start (so a span may overlap itself).  Returns ``(hist[S, cap] int32, len[S]
    int32, copied_fraction)``; slots beyond ``len`` hold -1.
    """
    cap = L if cap is None else cap
    cap = (cap + 3) // 4 * 4
    assert cap >= L
    cdf = zipf_cdf(V, s)
    perm = stream(seed, name + "/perm").permutation(V).astype(np.int32)
    lo, hi = span
    m = 0.5 * (lo + hi)
    pi = copy_frac / (copy_frac + m * (1.0 - copy_frac)) if copy_frac > 0 else 0.0
    hist = np.full((S, cap), -1, dtype=np.int32)
    copied = 0
    for si in range(S):
        g = stream(seed, f"{name}/{si}")
        n_ev = L  # upper bound on the number of events
        is_copy = g.random(n_ev) < pi
        is_copy[0] = False
        lens = np.where(is_copy, g.integers(lo, hi + 1, n_ev), 1).astype(np.int64)
        start = np.cumsum(lens) - lens            # position where each event begins
        keep = start < L
        is_copy, lens, start = is_copy[keep], lens[keep], start[keep]
        u = g.random(len(start))
        src0 = np.floor(u * start).astype(np.int64)   # uniform in [0, start)
        # per-position pointer: -1 for a fresh token, else the earlier position copied
        ptr = np.full(L, -1, dtype=np.int64)
        ev_of_pos = np.repeat(np.arange(len(start)), lens)[:L]
        off = np.arange(L) - start[ev_of_pos]
        cp = is_copy[ev_of_pos]
        ptr[cp] = src0[ev_of_pos][cp] + off[cp]
        fresh = _zipf_tokens(g, L, cdf, perm)
        root = np.where(ptr < 0, np.arange(L), ptr)
        while True:                                # pointer jumping to the fresh ancestor
            nxt = root[root]
            if np.array_equal(nxt, root):
                break
            root = nxt
        hist[si, :L] = fresh[root]
        copied += int(cp.sum())
    lens_out = np.full(S, L, dtype=np.int32)
    return hist, lens_out, copied / float(max(1, S * L))


# ----------------------------------------------------------------------------- hidden states
def hidden_literal(M: int, d: int, seed: int, name: str = "H") -> np.ndarray:
    """``[M, d]`` bf16 bits ~ N(0, 1)."""
    return f32_to_bf16_bits(stream(seed, name).standard_normal((M, d), dtype=np.float32))


def hidden_planted(W_bits: np.ndarray, targets: np.ndarray, seed: int, gain: float = 16.0,
                   name: str = "Hplant") -> np.ndarray:
    """Hidden states whose LM-head argmax is the given target token by a wide margin.

    Row m is ``gain * W[t_m] / |W[t_m]| + N(0, 1)``, rounded to bf16.
    """
    t = np.asarray(targets).reshape(-1)
    w = bf16_bits_to_f32(W_bits[t]).astype(np.float64)
    n = np.sqrt((w * w).sum(axis=1, keepdims=True))
    n[n == 0] = 1.0
    noise = stream(seed, name).standard_normal(w.shape, dtype=np.float32)
    return f32_to_bf16_bits((gain * w / n + noise).astype(np.float32))


def planted_targets(drafts: np.ndarray, n_drafts: np.ndarray, last_tokens: np.ndarray, V: int,
                    zipf_s: float, rho: float, seed: int, name: str = "plant"):
    """Choose the token each verify position should predict.

    ``drafts[S, B, w]``.  Per sequence one valid draft row r is picked uniformly and
    an accepted length a = min(w, G) with P(G >= j) = rho^j.  Targets for row r,
    positions j < a, equal the drafted token; position a gets a token different from
    the drafted one; every other position gets a random Zipf token.  Returns
    ``(targets[S, B, w+1] int32, row[S], a[S])``.
    """
    S, B, w = drafts.shape
    g = stream(seed, name)
    cdf = zipf_cdf(V, zipf_s)
    perm = stream(seed, name + "/perm").permutation(V).astype(np.int32)
    targets = _zipf_tokens(g, S * B * (w + 1), cdf, perm).reshape(S, B, w + 1)
    rows = np.zeros(S, dtype=np.int32)
    acc = np.zeros(S, dtype=np.int32)
    for s in range(S):
        nd = int(n_drafts[s])
        if nd <= 0:
            continue
        r = int(g.integers(0, nd))
        G = 0
        while G < w and g.random() < rho:
            G += 1
        rows[s], acc[s] = r, G
        targets[s, r, :G] = drafts[s, r, :G]
        if G < w:
            t = int(targets[s, r, G])
            if t == int(drafts[s, r, G]):
                t = (t + 1) % V
            targets[s, r, G] = t
    return targets.astype(np.int32), rows, acc


# ----------------------------------------------------------------------------- named workloads
CONFIGS = {
    # name: vocabulary V, hidden d, sequences S, history L, query lengths qs (priority order),
    #       rows per context strategy topk, draft rows B, draft width w, table width k_tab,
    #       weight dtype/std, Zipf exponent, copied-span fraction, seed
    "C1": dict(V=1024, d=128, S=1, L=512, qs=(1,), topk=4, B=4, w=4, k_tab=4,
               wdtype="f32", wstd=128 ** -0.5, zipf=1.1, copy=0.20, seed=0),
    "C2": dict(V=32000, d=4096, S=1, L=4096, qs=(2, 1), topk=8, B=8, w=5, k_tab=8,
               wdtype="bf16", wstd=0.02, zipf=1.1, copy=0.20, seed=1),
    "C3": dict(V=32000, d=4096, S=64, L=2048, qs=(3, 2, 1), topk=4, B=16, w=8, k_tab=8,
               wdtype="bf16", wstd=0.02, zipf=1.1, copy=0.30, seed=2),
    "C4": dict(V=128256, d=4096, S=8, L=8192, qs=(2,), topk=32, B=32, w=6, k_tab=10,
               wdtype="bf16", wstd=0.02, zipf=1.1, copy=0.20, seed=3),
    "C5": dict(V=128256, d=4096, S=4, L=131072, qs=(3, 2), topk=8, B=64, w=10, k_tab=10,
               wdtype="bf16", wstd=0.02, zipf=1.05, copy=0.40, seed=4),
}


def config(name: str) -> dict:
    c = dict(CONFIGS[name])
    c["name"] = name
    # C3 reuses C2's head (and table), C5 reuses C4's: weights are keyed by wseed
    c["wseed"] = {"C3": CONFIGS["C2"]["seed"], "C5": CONFIGS["C4"]["seed"]}.get(name, c["seed"])
    c["M"] = c["S"] * c["B"] * (c["w"] + 1)
    return c
