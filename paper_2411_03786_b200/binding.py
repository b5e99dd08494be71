"""ctypes binding of ``include/ngram_spec.h``: same names, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
import re

import torch

from .build import LIB, build_library

FLAG_DEDUP, FLAG_MODEL_FILL, FLAG_KEY_NEXT_TOKEN, FLAG_PARTIAL_TAIL = 1, 2, 4, 8
STATUS_TOKEN_RANGE, STATUS_CAPACITY, STATUS_TIMEOUT, STATUS_GROUPS, STATUS_INDEX = 1, 2, 4, 8, 16
SPEC_F32, SPEC_BF16 = 0, 1

_HEADER = os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", "include", "ngram_spec.h")
_lib = None


def flag_reserve(n: int) -> int:
    """Draft flag bits that reserve ``n`` rows for the model strategy (SPEC_FLAG_RESERVE)."""
    return (int(n) & 0xFF) << 8


class SpecError(RuntimeError):
    pass


def declared_symbols() -> list[str]:
    """Function names declared in the public header."""
    text = re.sub(r"/\*.*?\*/", "", open(_HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b([a-z_][a-z0-9_]*)\s*\(", text)) - {"defined"})


def load_library(build: bool = True) -> C.CDLL:
    """Load (building first if needed) the CUDA library.  Fails loudly if it cannot be loaded."""
    global _lib
    if _lib is not None:
        return _lib
    if build:
        build_library()
    if not os.path.exists(LIB):
        raise SpecError(f"{LIB} is missing: build it with `python -m paper_2411_03786_b200.build`")
    lib = C.CDLL(LIB)
    vp, ip, i32p, fp = C.c_void_p, C.POINTER(C.c_int), C.c_void_p, C.c_void_p
    lib.spec_init.argtypes = [C.POINTER(vp), vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp]
    lib.spec_destroy.argtypes = [vp]
    lib.spec_get_status.argtypes = [vp, ip, vp]
    lib.spec_last_error.argtypes = [vp]
    lib.spec_last_error.restype = C.c_char_p
    lib.build_model_ngram_tables.argtypes = [vp, vp, C.c_int, C.c_int, i32p, fp, i32p, vp]
    lib.build_model_unigram.argtypes = [vp, C.c_int, i32p, fp, vp]
    lib.spec_set_model_table.argtypes = [vp, i32p, C.c_int, i32p, C.c_int]
    lib.draft_context_ngrams.argtypes = [vp, i32p, i32p, C.c_int, C.c_int, ip, C.c_int, C.c_int, C.c_int, C.c_int,
                                         C.c_int, i32p, i32p, i32p, i32p, vp]
    lib.verify_lmhead_argmax.argtypes = [vp, vp, C.c_int, i32p, fp, vp]
    lib.accept_and_commit.argtypes = [vp, i32p, i32p, i32p, C.c_int, C.c_int, C.c_int, i32p, i32p, C.c_int, i32p,
                                      i32p, i32p, vp]
    lib.verify_accept_commit.argtypes = [vp, vp, i32p, i32p, C.c_int, C.c_int, C.c_int, i32p, i32p, i32p, C.c_int, i32p,
                                         i32p, i32p, vp]
    lib.verify_lmhead_keys.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp]
    lib.spec_unpack_keys.argtypes = [vp, C.c_int, C.c_int, i32p, fp, vp]
    lib.spec_accumulate_stats.argtypes = [vp, i32p, i32p, i32p, C.c_int, C.c_int, C.c_int, vp, vp]
    lib.spec_debug_logits.argtypes = [vp, vp, C.c_int, fp, vp]
    lib.spec_quantize_rows_fp8.argtypes = [vp, vp, C.c_int, vp, fp, vp]
    lib.spec_quantize_head_fp8.argtypes = [vp, vp, fp, vp]
    lib.spec_set_head_fp8.argtypes = [vp, vp, fp]
    lib.verify_lmhead_argmax_fp8.argtypes = [vp, vp, C.c_int, vp, fp, i32p, fp, vp]
    lib.verify_lmhead_argmax_noalloc.argtypes = [vp, C.c_int, C.c_int, vp, C.c_int, i32p, fp, C.c_int, vp]
    lib.build_model_ngram_table_rows.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, i32p, fp, vp]
    lib.spec_extend_model_table.argtypes = [vp, i32p, C.c_int, C.c_int, i32p, vp]
    lib.spec_debug_expire_wait.argtypes = [vp, C.c_ulonglong, C.c_int, vp]
    lib.spec_context_index_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
    lib.spec_context_index_bytes.restype = C.c_size_t
    lib.spec_context_index_build.argtypes = [vp, vp, i32p, i32p, C.c_int, C.c_int, ip, C.c_int, C.c_int, C.c_int, vp]
    lib.draft_context_ngrams_indexed.argtypes = [vp, vp, i32p, i32p, C.c_int, C.c_int, ip, C.c_int, C.c_int, C.c_int, C.c_int,
                                                 C.c_int, i32p, i32p, i32p, i32p, vp]
    lib.accept_and_commit_indexed.argtypes = [vp, vp, i32p, i32p, i32p, C.c_int, C.c_int, C.c_int, i32p, i32p, C.c_int, i32p,
                                              i32p, i32p, vp]
    lib.spec_launch_count.argtypes = [vp]
    lib.spec_launch_count.restype = C.c_longlong
    _lib = lib
    return lib


def _ptr(t, dtype=None):
    if t is None:
        return None
    # pinned host memory is mapped into the device address space (unified addressing): small outputs may
    # live there so that a kernel's result reaches the host without a separate copy
    assert (t.is_cuda or t.is_pinned()) and t.is_contiguous(), "tensors must be contiguous CUDA (or pinned host) tensors"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class SpecContext:
    """One model head on one GPU.  Methods mirror the C entry points and launch on torch's current stream."""

    def __init__(self, embed: torch.Tensor, unembed: torch.Tensor):
        self._lib = load_library()
        self._h = C.c_void_p()
        if not torch.cuda.is_available():
            raise SpecError("no CUDA device: this library has no CPU path")
        assert embed.shape == unembed.shape and embed.dtype == unembed.dtype
        dtype = {torch.float32: SPEC_F32, torch.bfloat16: SPEC_BF16}[embed.dtype]
        self.V, self.d = int(embed.shape[0]), int(embed.shape[1])
        self._keep = [embed, unembed]
        rc = self._lib.spec_init(C.byref(self._h), _ptr(embed), _ptr(unembed), dtype, self.V, self.d,
                                 embed.device.index or 0, _stream())
        if rc != 0:
            raise SpecError(f"spec_init failed ({rc}): {self._lib.spec_last_error(None).decode()}")

    def _check(self, rc: int, what: str):
        if rc != 0:
            raise SpecError(f"{what} failed ({rc}): {self._lib.spec_last_error(self._h).decode()}")

    def close(self):
        if self._h:
            torch.cuda.synchronize()
            self._lib.spec_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def get_status(self) -> int:
        bits = C.c_int(0)
        self._check(self._lib.spec_get_status(self._h, C.byref(bits), _stream()), "spec_get_status")
        return bits.value

    def launch_count(self) -> int:
        return int(self._lib.spec_launch_count(self._h))

    def build_model_ngram_tables(self, k_tab: int, rows: torch.Tensor | None = None, w_ext: int = 0,
                                 with_values: bool = False):
        dev = self._keep[0].device
        tab = torch.empty((self.V, k_tab), dtype=torch.int32, device=dev)
        val = torch.empty((self.V, k_tab), dtype=torch.float32, device=dev) if with_values else None
        ext = torch.empty((self.V, k_tab, w_ext), dtype=torch.int32, device=dev) if w_ext > 0 else None
        self._check(self._lib.build_model_ngram_tables(self._h, _ptr(rows, torch.bfloat16), k_tab, w_ext, _ptr(tab),
                                                       _ptr(val), _ptr(ext), _stream()), "build_model_ngram_tables")
        self._keep_table = (tab, ext, rows)
        return tab, val, ext

    def build_model_ngram_table_rows(self, k_tab: int, row_begin: int, row_count: int, tab: torch.Tensor,
                                     val: torch.Tensor | None = None, rows: torch.Tensor | None = None):
        """Writes rows ``[row_begin, row_begin + row_count)`` of the whole ``tab[V, k_tab]`` (one rank's slice)."""
        assert tuple(tab.shape) == (self.V, k_tab)
        self._check(self._lib.build_model_ngram_table_rows(self._h, _ptr(rows, torch.bfloat16), int(row_begin), int(row_count),
                                                           k_tab, _ptr(tab, torch.int32), _ptr(val, torch.float32), _stream()),
                    "build_model_ngram_table_rows")
        return tab

    def extend_model_table(self, tab: torch.Tensor, w_ext: int):
        """Extension ``ext[V, k_tab, w_ext]`` of a complete table; adopts both for drafting."""
        k_tab = int(tab.shape[1])
        ext = torch.empty((self.V, k_tab, w_ext), dtype=torch.int32, device=tab.device)
        self._check(self._lib.spec_extend_model_table(self._h, _ptr(tab, torch.int32), k_tab, int(w_ext), _ptr(ext), _stream()),
                    "spec_extend_model_table")
        self._keep_table = (tab, ext, None)
        return ext

    def debug_expire_wait(self, limit_ns: int = 20000, mark_verify_incomplete: bool = False):
        self._check(self._lib.spec_debug_expire_wait(self._h, int(limit_ns), int(mark_verify_incomplete), _stream()),
                    "spec_debug_expire_wait")

    def build_model_unigram(self, k_uni: int):
        """Returns ``(ids[k_uni] by ascending distance, dist2[V])``."""
        dev = self._keep[0].device
        idx = torch.empty(max(k_uni, 1), dtype=torch.int32, device=dev)
        dist2 = torch.empty(self.V, dtype=torch.float32, device=dev)
        self._check(self._lib.build_model_unigram(self._h, k_uni, _ptr(idx), _ptr(dist2), _stream()), "build_model_unigram")
        return idx[:k_uni], dist2

    def set_model_table(self, tab: torch.Tensor, ext: torch.Tensor | None = None):
        k_tab = int(tab.shape[1])
        w_ext = int(ext.shape[2]) if ext is not None else 0
        self._check(self._lib.spec_set_model_table(self._h, _ptr(tab, torch.int32), k_tab, _ptr(ext, torch.int32), w_ext),
                    "spec_set_model_table")
        self._keep_table = (tab, ext, None)

    def draft_context_ngrams(self, hist: torch.Tensor, lens: torch.Tensor, qs, topk: int, B: int, w: int,
                             flags: int = FLAG_DEDUP | FLAG_MODEL_FILL, out=None):
        S, cap = int(hist.shape[0]), int(hist.shape[1])
        dev = hist.device
        if out is None:
            out = (torch.empty((S, B, w), dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
                   torch.empty((S, B), dtype=torch.int32, device=dev), torch.empty((S, B), dtype=torch.int32, device=dev))
        drafts, nd, src, counts = out
        qs_arr = (C.c_int * max(1, len(qs)))(*[int(q) for q in qs])
        self._check(self._lib.draft_context_ngrams(self._h, _ptr(hist, torch.int32), _ptr(lens, torch.int32), S, cap,
                                                   qs_arr, len(qs), topk, B, w, flags, _ptr(drafts), _ptr(nd),
                                                   _ptr(src), _ptr(counts), _stream()), "draft_context_ngrams")
        return drafts, nd, src, counts

    def context_index_build(self, hist: torch.Tensor, lens: torch.Tensor, qs, w: int, flags: int = 0, index: torch.Tensor | None = None):
        """Builds (and registers) the incremental context index of the current histories; returns the index buffer."""
        S, cap = int(hist.shape[0]), int(hist.shape[1])
        need = int(self._lib.spec_context_index_bytes(S, cap, len(qs)))
        if index is None:
            index = torch.empty(need, dtype=torch.uint8, device=hist.device)
        assert index.numel() >= need
        qs_arr = (C.c_int * max(1, len(qs)))(*[int(q) for q in qs])
        self._check(self._lib.spec_context_index_build(self._h, _ptr(index), _ptr(hist, torch.int32), _ptr(lens, torch.int32), S, cap,
                                                       qs_arr, len(qs), w, flags, _stream()), "spec_context_index_build")
        self._keep_index = index
        return index

    def draft_context_ngrams_indexed(self, index: torch.Tensor, hist: torch.Tensor, lens: torch.Tensor, qs, topk: int, B: int, w: int,
                                     flags: int = FLAG_DEDUP | FLAG_MODEL_FILL, out=None):
        S, cap = int(hist.shape[0]), int(hist.shape[1])
        dev = hist.device
        if out is None:
            out = (torch.empty((S, B, w), dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
                   torch.empty((S, B), dtype=torch.int32, device=dev), torch.empty((S, B), dtype=torch.int32, device=dev))
        drafts, nd, src, counts = out
        qs_arr = (C.c_int * max(1, len(qs)))(*[int(q) for q in qs])
        self._check(self._lib.draft_context_ngrams_indexed(self._h, _ptr(index), _ptr(hist, torch.int32), _ptr(lens, torch.int32), S, cap,
                                                           qs_arr, len(qs), topk, B, w, flags, _ptr(drafts), _ptr(nd),
                                                           _ptr(src), _ptr(counts), _stream()), "draft_context_ngrams_indexed")
        return drafts, nd, src, counts

    def accept_and_commit_indexed(self, index: torch.Tensor, drafts, n_drafts, argmax, hist, lens, out=None):
        S, B, w = (int(x) for x in drafts.shape)
        cap = int(hist.shape[1])
        dev = hist.device
        if out is None:
            out = (torch.empty(S, dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
                   torch.empty((S, w + 1), dtype=torch.int32, device=dev))
        acc, best, com = out
        self._check(self._lib.accept_and_commit_indexed(self._h, _ptr(index), _ptr(drafts, torch.int32), _ptr(n_drafts, torch.int32),
                                                        _ptr(argmax, torch.int32), S, B, w, _ptr(hist, torch.int32),
                                                        _ptr(lens, torch.int32), cap, _ptr(acc), _ptr(best), _ptr(com),
                                                        _stream()), "accept_and_commit_indexed")
        return acc, best, com

    def verify_lmhead_argmax(self, hidden: torch.Tensor, out=None, with_max: bool = False):
        M = int(hidden.shape[0])
        if out is None:
            out = (torch.empty(M, dtype=torch.int32, device=hidden.device),
                   torch.empty(M, dtype=torch.float32, device=hidden.device) if with_max else None)
        am, mx = out
        self._check(self._lib.verify_lmhead_argmax(self._h, _ptr(hidden, torch.bfloat16), M, _ptr(am), _ptr(mx),
                                                   _stream()), "verify_lmhead_argmax")
        return am, mx

    def accept_and_commit(self, drafts, n_drafts, argmax, hist, lens, out=None):
        S, B, w = (int(x) for x in drafts.shape)
        cap = int(hist.shape[1])
        dev = hist.device
        if out is None:
            out = (torch.empty(S, dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
                   torch.empty((S, w + 1), dtype=torch.int32, device=dev))
        acc, best, com = out
        self._check(self._lib.accept_and_commit(self._h, _ptr(drafts, torch.int32), _ptr(n_drafts, torch.int32),
                                                _ptr(argmax, torch.int32), S, B, w, _ptr(hist, torch.int32),
                                                _ptr(lens, torch.int32), cap, _ptr(acc), _ptr(best), _ptr(com),
                                                _stream()), "accept_and_commit")
        return acc, best, com

    def verify_accept_commit(self, hidden, drafts, n_drafts, hist, lens, argmax=None, out=None):
        """Fused verify + accept: returns ``(argmax[S, B, w+1], acc_len, best_row, committed)``."""
        S, B, w = (int(x) for x in drafts.shape)
        cap = int(hist.shape[1])
        dev = hist.device
        if argmax is None:
            argmax = torch.empty(S * B * (w + 1), dtype=torch.int32, device=dev)
        if out is None:
            out = (torch.empty(S, dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
                   torch.empty((S, w + 1), dtype=torch.int32, device=dev))
        acc, best, com = out
        self._check(self._lib.verify_accept_commit(self._h, _ptr(hidden, torch.bfloat16), _ptr(drafts, torch.int32),
                                                   _ptr(n_drafts, torch.int32), S, B, w, _ptr(argmax, torch.int32),
                                                   _ptr(hist, torch.int32), _ptr(lens, torch.int32), cap, _ptr(acc),
                                                   _ptr(best), _ptr(com), _stream()), "verify_accept_commit")
        return argmax.view(S, B, w + 1), acc, best, com

    def verify_lmhead_keys(self, hidden: torch.Tensor, vocab_offset: int, keys: torch.Tensor | None = None):
        """Per-row (logit, global id) keys of this context's vocabulary shard, as sortable int64."""
        M = int(hidden.shape[0])
        if keys is None:
            keys = torch.empty(M, dtype=torch.int64, device=hidden.device)
        self._check(self._lib.verify_lmhead_keys(self._h, _ptr(hidden, torch.bfloat16), M, int(vocab_offset),
                                                 _ptr(keys, torch.int64), _stream()), "verify_lmhead_keys")
        return keys

    def accumulate_stats(self, acc_len, best_row, src, w: int, stats: torch.Tensor | None = None):
        """Adds one step to the ablation histograms ([w+1] | [B] | [5] | [5] int64)."""
        S, B = int(src.shape[0]), int(src.shape[1])
        if stats is None:
            stats = torch.zeros((w + 1) + B + 10, dtype=torch.int64, device=src.device)
        self._check(self._lib.spec_accumulate_stats(self._h, _ptr(acc_len, torch.int32), _ptr(best_row, torch.int32),
                                                    _ptr(src, torch.int32), S, B, w, _ptr(stats, torch.int64), _stream()),
                    "spec_accumulate_stats")
        return stats

    def quantize_rows_fp8(self, rows: torch.Tensor, out=None):
        """Per-row E4M3 quantisation of a bf16 matrix: ``(codes uint8 [n, d], scale float32 [n])``."""
        n = int(rows.shape[0])
        if out is None:
            out = (torch.empty((n, self.d), dtype=torch.uint8, device=rows.device),
                   torch.empty(n, dtype=torch.float32, device=rows.device))
        codes, scale = out
        self._check(self._lib.spec_quantize_rows_fp8(self._h, _ptr(rows, torch.bfloat16), n, _ptr(codes, torch.uint8),
                                                     _ptr(scale, torch.float32), _stream()), "spec_quantize_rows_fp8")
        return codes, scale

    def quantize_head_fp8(self):
        """Builds (and adopts) the 8-bit copy of the unembedding: ``(codes uint8 [V, d], scale float32 [V])``."""
        dev = self._keep[0].device
        wq = torch.empty((self.V, self.d), dtype=torch.uint8, device=dev)
        ws = torch.empty(self.V, dtype=torch.float32, device=dev)
        self._check(self._lib.spec_quantize_head_fp8(self._h, _ptr(wq), _ptr(ws), _stream()), "spec_quantize_head_fp8")
        self._keep_fp8 = (wq, ws)
        return wq, ws

    def set_head_fp8(self, wq: torch.Tensor, ws: torch.Tensor):
        self._check(self._lib.spec_set_head_fp8(self._h, _ptr(wq, torch.uint8), _ptr(ws, torch.float32)), "spec_set_head_fp8")
        self._keep_fp8 = (wq, ws)

    def verify_lmhead_argmax_fp8(self, hidden: torch.Tensor | None, scratch=None, out=None, with_max: bool = False):
        """``scratch = (codes uint8 [M, d], scale float32 [M])`` receives the quantised hidden states; with
        ``hidden=None`` it already holds them."""
        M = int(hidden.shape[0]) if hidden is not None else int(scratch[0].shape[0])
        dev = hidden.device if hidden is not None else scratch[0].device
        if scratch is None:
            scratch = (torch.empty((M, self.d), dtype=torch.uint8, device=dev), torch.empty(M, dtype=torch.float32, device=dev))
        if out is None:
            out = (torch.empty(M, dtype=torch.int32, device=dev),
                   torch.empty(M, dtype=torch.float32, device=dev) if with_max else None)
        am, mx = out
        self._check(self._lib.verify_lmhead_argmax_fp8(self._h, _ptr(hidden, torch.bfloat16), M, _ptr(scratch[0], torch.uint8),
                                                       _ptr(scratch[1], torch.float32), _ptr(am), _ptr(mx), _stream()),
                    "verify_lmhead_argmax_fp8")
        return am, mx

    def debug_logits(self, rows: torch.Tensor) -> torch.Tensor:
        m = int(rows.shape[0])
        out = torch.empty((m, self.V), dtype=torch.float32, device=rows.device)
        self._check(self._lib.spec_debug_logits(self._h, _ptr(rows, torch.bfloat16), m, _ptr(out), _stream()),
                    "spec_debug_logits")
        return out


def verify_lmhead_argmax_noalloc(unembed: torch.Tensor, hidden: torch.Tensor, out):
    """Context-free verification for callers that must not allocate device memory.

    ``out = (argmax int32 [M], max float32 [M] or None)`` must be preallocated by the caller: this
    wrapper allocates nothing either.  See ``verify_lmhead_argmax_noalloc`` in the header for the
    row limit and the rule that calls must not overlap on the GPU.
    """
    lib = load_library()
    am, mx = out
    V, d = int(unembed.shape[0]), int(unembed.shape[1])
    rc = lib.verify_lmhead_argmax_noalloc(_ptr(unembed, torch.bfloat16), V, d, _ptr(hidden, torch.bfloat16),
                                          int(hidden.shape[0]), _ptr(am, torch.int32), _ptr(mx), unembed.device.index or 0,
                                          _stream())
    if rc != 0:
        raise SpecError(f"verify_lmhead_argmax_noalloc failed ({rc}): {lib.spec_last_error(None).decode()}")
    return am, mx


def unpack_keys(keys: torch.Tensor, V_total: int, with_max: bool = False):
    """Token ids (and winning logits) from merged shard keys."""
    lib = load_library()
    M = int(keys.shape[0])
    am = torch.empty(M, dtype=torch.int32, device=keys.device)
    mx = torch.empty(M, dtype=torch.float32, device=keys.device) if with_max else None
    rc = lib.spec_unpack_keys(_ptr(keys, torch.int64), M, int(V_total), _ptr(am), _ptr(mx), _stream())
    if rc != 0:
        raise SpecError(f"spec_unpack_keys failed ({rc}): {lib.spec_last_error(None).decode()}")
    return am, mx
