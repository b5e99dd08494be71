"""Pins for the oracle's context N-gram (Section 4.2) against things other than itself."""
import collections
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def brute_context(hist, q, w, topk):
    """Independent restatement with a dict keyed by the continuation tuple."""
    hist = list(int(t) for t in hist)
    L = len(hist)
    if L < q + w:
        return []
    query = tuple(hist[L - q:])
    groups = {}
    for i in range(0, L - q - w + 1):
        if tuple(hist[i:i + q]) == query:
            c = tuple(hist[i + q:i + q + w])
            cnt, last = groups.get(c, (0, -1))
            groups[c] = (cnt + 1, max(last, i))
    order = sorted(groups.items(), key=lambda kv: (-kv[1][0], -kv[1][1]))
    return [(c, cnt, last) for c, (cnt, last) in order[:topk]]


def as_list(res):
    rows, counts, lasts = res
    return [(tuple(int(t) for t in r), int(c), int(l)) for r, c, l in zip(rows, counts, lasts)]


def test_hand_example_from_golden_file():
    hist = q = w = None
    rows = []
    for line in open(os.path.join(GOLD, "context_hand_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(" ", 1)
        if key == "hist":
            hist = [int(t) for t in rest.split()]
        elif key == "q":
            q = int(rest)
        elif key == "w":
            w = int(rest)
        elif key == "row":
            toks, cnt, last = rest.split("|")
            rows.append((tuple(int(t) for t in toks.split()), int(cnt), int(last)))
    assert as_list(oracle.context_draft(hist, q, w, 3)) == rows
    assert as_list(oracle.context_draft(hist, q, w, 2)) == rows[:2]
    assert as_list(oracle.context_draft(hist, q, w, 8)) == rows


@pytest.mark.parametrize("vocab", [2, 3, 4])
def test_brute_force_on_tiny_histories_with_many_ties(vocab):
    g = np.random.default_rng(100 + vocab)
    for trial in range(300):
        L = int(g.integers(0, 65))
        q = int(g.integers(1, 5))
        w = int(g.integers(1, 5))
        topk = int(g.integers(1, 9))
        hist = g.integers(0, vocab, L).astype(np.int32)
        assert as_list(oracle.context_draft(hist, q, w, topk)) == brute_context(hist, q, w, topk), (L, q, w, topk)


def test_library_unique_gives_the_same_groups_and_counts():
    # numpy's sliding windows + unique(axis=0) restate "count each distinct (q+w)-gram
    # whose first q tokens equal the query" with library routines.
    g = np.random.default_rng(7)
    for trial in range(50):
        L, q, w = int(g.integers(8, 400)), int(g.integers(1, 4)), int(g.integers(1, 6))
        hist = g.integers(0, 6, L).astype(np.int32)
        win = np.lib.stride_tricks.sliding_window_view(hist, q + w)
        m = win[(win[:, :q] == hist[L - q:]).all(axis=1)]
        rows, counts, _ = oracle.context_draft(hist, q, w, topk=10 ** 6)
        if len(m) == 0:
            assert len(rows) == 0
            continue
        u, c = np.unique(m[:, q:], axis=0, return_counts=True)
        want = collections.Counter({tuple(r): int(n) for r, n in zip(u.tolist(), c.tolist())})
        got = collections.Counter({tuple(r): int(n) for r, n in zip(rows.tolist(), counts.tolist())})
        assert got == want
        assert sum(got.values()) == len(m)


def test_invariants():
    # constant history: one group holding every eligible window
    L, q, w = 50, 2, 3
    rows, counts, lasts = oracle.context_draft(np.full(L, 9, np.int32), q, w, 4)
    assert rows.tolist() == [[9, 9, 9]] and counts.tolist() == [L - q - w + 1] and lasts.tolist() == [L - q - w]
    # q = w = 1 is the next-token histogram of the last token (excluding the final position)
    g = np.random.default_rng(3)
    hist = g.integers(0, 5, 200).astype(np.int32)
    nxt = collections.Counter(int(hist[i + 1]) for i in range(len(hist) - 1) if hist[i] == hist[-1])
    rows, counts, _ = oracle.context_draft(hist, 1, 1, 100)
    assert {int(r[0]): int(c) for r, c in zip(rows, counts)} == dict(nxt)
    assert all(counts[i] >= counts[i + 1] for i in range(len(counts) - 1))
    # relabelling the vocabulary relabels the output and nothing else
    perm = g.permutation(5).astype(np.int32)
    r2, c2, l2 = oracle.context_draft(perm[hist], 1, 1, 100)
    assert np.array_equal(r2, perm[rows]) and np.array_equal(c2, counts)
    # too short for one full window -> nothing
    assert len(oracle.context_draft(np.array([1, 1, 1], np.int32), 2, 2, 4)[0]) == 0
    assert len(oracle.context_draft(np.array([], np.int32), 1, 1, 4)[0]) == 0
    # exactly one full window
    r, c, l = oracle.context_draft(np.array([1, 2, 3, 1], np.int32), 1, 2, 4)
    assert r.tolist() == [[2, 3]] and c.tolist() == [1] and l.tolist() == [0]


def test_later_occurrence_wins_ties_and_count_wins_over_recency():
    #            0  1  2  3  4  5  6  7  8  9 10
    hist = [4, 1, 4, 2, 4, 1, 4, 3, 4, 2, 4]
    rows, counts, lasts = oracle.context_draft(np.array(hist, np.int32), 1, 1, 3)
    # after 4: 1 (x2, last 4), 2 (x2, last 8), 3 (x1, last 6); window 10 has no continuation
    assert rows.reshape(-1).tolist() == [2, 1, 3] and counts.tolist() == [2, 2, 1] and lasts.tolist() == [8, 4, 6]


def test_next_token_keyed_variant():
    g = np.random.default_rng(21)
    for trial in range(100):
        L, q, w = int(g.integers(0, 80)), int(g.integers(1, 4)), int(g.integers(1, 5))
        hist = g.integers(0, 3, L).astype(np.int32)
        rows, counts, lasts = oracle.context_draft(hist, q, w, 10, key_len=1)
        if L < q + w:
            assert len(rows) == 0
            continue
        # counts are the histogram of the token right after each eligible occurrence of the query
        nxt, last = collections.Counter(), {}
        for i in range(L - q - w + 1):
            if (hist[i:i + q] == hist[L - q:]).all():
                t = int(hist[i + q])
                nxt[t] += 1
                last[t] = i
        order = sorted(nxt, key=lambda t: (-nxt[t], -last[t]))[:10]
        assert [int(r[0]) for r in rows] == order
        assert counts.tolist() == [nxt[t] for t in order] and lasts.tolist() == [last[t] for t in order]
        for r, l in zip(rows, lasts):                         # the row is what followed the latest occurrence
            assert r.tolist() == hist[l + q:l + q + w].tolist()
    # with w = 1 the variant and the paper's rule coincide
    hist = g.integers(0, 4, 60).astype(np.int32)
    a = oracle.context_draft(hist, 1, 1, 8)
    b = oracle.context_draft(hist, 1, 1, 8, key_len=1)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


# ----------------------------------------------------------------------------- partial continuations near the tail
def brute_context_partial(hist, q, w, topk, key_len=None):
    """Dictionary restatement: every occurrence of the last q tokens that has at least one token after it; a
    continuation that runs past the end of the history repeats the tokens it has."""
    hist = [int(t) for t in hist]
    L = len(hist)
    key_len = w if key_len is None else key_len
    if L < q + 1:
        return []
    groups = {}
    for i in range(L - q):
        if hist[i:i + q] != hist[L - q:]:
            continue
        p = i + q
        have = hist[p:]
        cont = tuple(have[t] if t < len(have) else have[t % len(have)] for t in range(w))
        cnt, _, _ = groups.get(cont[:key_len], (0, -1, None))
        groups[cont[:key_len]] = (cnt + 1, i, cont)          # i increases: the latest occurrence supplies the row
    order = sorted(groups.values(), key=lambda v: (-v[0], -v[1]))[:topk]
    return [(cont, cnt, last) for cnt, last, cont in order]


def test_partial_tail_hand_example():
    # "1 2 3" repeats; the query is the final "1 2".  Full windows of 2 + 4 tokens: only the one at 0, continuation
    # 3 1 2 3.  The occurrence at 3 has three tokens after it (3 1 2); continued periodically it reads 3 1 2 3 as
    # well, so with partial continuations the same row is seen twice, the later time at window start 3.
    hist = np.array([1, 2, 3, 1, 2, 3, 1, 2], np.int32)
    rows, counts, lasts = oracle.context_draft(hist, 2, 4, 4)
    assert rows.tolist() == [[3, 1, 2, 3]] and counts.tolist() == [1] and lasts.tolist() == [0]
    rows, counts, lasts = oracle.context_draft_partial(hist, 2, 4, 4)
    assert rows.tolist() == [[3, 1, 2, 3]] and counts.tolist() == [2] and lasts.tolist() == [3]
    # one token after the occurrence: it alone is repeated
    hist = np.array([5, 7, 9, 4, 5, 7], np.int32)            # query "7"; occurrence at 1 is followed by 9 4 5 7 ...
    rows, counts, lasts = oracle.context_draft_partial(hist, 1, 6, 3)
    assert rows.tolist() == [[9, 4, 5, 7, 9, 4]] and counts.tolist() == [1]
    hist = np.array([8, 8, 8], np.int32)                      # query "8": occurrences at 0 (followed by 8 8) and 1 (by 8)
    rows, counts, lasts = oracle.context_draft_partial(hist, 1, 5, 3)
    assert rows.tolist() == [[8, 8, 8, 8, 8]] and counts.tolist() == [2] and lasts.tolist() == [1]


def test_partial_tail_against_brute_force():
    g = np.random.default_rng(21)
    for trial in range(900):
        A = int(g.integers(1, 4))
        L = int(g.integers(0, 40))
        hist = g.integers(0, A, L).astype(np.int32)
        if trial % 3 == 0 and L > 6:                          # periodic tails, where the extension matters most
            per = int(g.integers(1, 5))
            hist[L // 2:] = np.resize(hist[L // 2:L // 2 + per], L - L // 2)
        q, w, topk = int(g.integers(1, 5)), int(g.integers(1, 8)), int(g.integers(1, 6))
        key_len = 1 if trial % 4 == 0 else w
        want = brute_context_partial(hist, q, w, topk, key_len)
        rows, counts, lasts = oracle.context_draft_partial(hist, q, w, topk, key_len)
        assert rows.tolist() == [list(c) for c, _, _ in want]
        assert counts.tolist() == [n for _, n, _ in want] and lasts.tolist() == [i for _, _, i in want]


def test_partial_tail_reduces_to_the_plain_rule_when_no_occurrence_is_near_the_end():
    g = np.random.default_rng(22)
    for _ in range(200):
        L, q, w = int(g.integers(20, 60)), int(g.integers(1, 4)), int(g.integers(1, 7))
        hist = g.integers(0, 3, L).astype(np.int32)
        hist[L - q:] = 9                                       # the query occurs nowhere else ...
        pos = int(g.integers(0, L - q - w - q + 1)) if L - q - w - q + 1 > 0 else 0
        hist[pos:pos + q] = 9                                  # ... except once, far enough from the end
        a = oracle.context_draft(hist, q, w, 5)
        b = oracle.context_draft_partial(hist, q, w, 5)
        assert all(np.array_equal(x, y) for x, y in zip(a, b))
