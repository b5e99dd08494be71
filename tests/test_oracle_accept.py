"""Pins for the oracle's greedy acceptance, commit, mixing and table extension."""
import os

import numpy as np

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def brute_accept(drafts, nd, P, hist, lens):
    drafts, P, hist, lens = drafts.copy(), P.copy(), hist.copy(), lens.copy()
    S, B, w = drafts.shape
    cap = hist.shape[1]
    acc, best, com = [], [], []
    for s in range(S):
        lengths = []
        for b in range(int(nd[s])):
            n = 0
            for j in range(w):
                if drafts[s, b, j] != P[s, b, j]:
                    break
                n += 1
            lengths.append(n)
        if lengths:
            a = max(lengths)
            bb = lengths.index(a)
        else:
            a, bb = 0, 0
        toks = [int(t) for t in drafts[s, bb, :a]] + [int(P[s, bb, a])]
        if lens[s] + len(toks) > cap:
            acc.append(-1); best.append(-1); com.append([-1] * (w + 1))
            continue
        hist[s, lens[s]:lens[s] + len(toks)] = toks
        lens[s] += len(toks)
        acc.append(a); best.append(bb); com.append(toks + [-1] * (w + 1 - len(toks)))
    return np.array(acc), np.array(best), np.array(com), hist, lens


def test_hand_example_from_golden_file():
    d, p, exp = [], [], {}
    for line in open(os.path.join(GOLD, "accept_hand_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(" ", 1)
        vals = [int(t) for t in rest.split()]
        if key == "draft":
            d.append(vals)
        elif key == "pred":
            p.append(vals)
        else:
            exp[key] = vals
    drafts = np.array([d], np.int32)
    P = np.array([p], np.int32)
    hist = np.full((1, 8), -1, np.int32)
    hist[0, :2] = [1, 5]
    lens = np.array([2], np.int32)
    acc, best, com = oracle.accept_commit(drafts, np.array([3], np.int32), P, hist, lens)
    assert acc.tolist() == [max(exp["accepted"])] and best.tolist() == exp["best"]
    assert com[0].tolist() == exp["committed"]
    assert hist[0].tolist() == [1, 5] + exp["committed"] + [-1] * 3 and lens.tolist() == [5]
    # each row on its own reproduces the per-row accepted lengths
    for b, a in enumerate(exp["accepted"]):
        h = np.full((1, 8), -1, np.int32)
        acc1, _, _ = oracle.accept_commit(drafts[:, b:b + 1], np.array([1], np.int32), P[:, b:b + 1], h,
                                          np.array([0], np.int32))
        assert acc1.tolist() == [a]


def test_brute_force_small_alphabet():
    g = np.random.default_rng(11)
    for trial in range(200):
        S, B, w = int(g.integers(1, 5)), int(g.integers(1, 7)), int(g.integers(1, 6))
        A = int(g.integers(2, 4))
        drafts = g.integers(0, A, (S, B, w)).astype(np.int32)
        P = g.integers(0, A, (S, B, w + 1)).astype(np.int32)
        nd = g.integers(0, B + 1, S).astype(np.int32)
        cap = 12
        lens = g.integers(0, cap + 1, S).astype(np.int32)   # some sequences cannot take the commit
        hist = np.full((S, cap), -1, np.int32)
        for s in range(S):
            hist[s, :lens[s]] = g.integers(0, A, lens[s])
        e_acc, e_best, e_com, e_hist, e_lens = brute_accept(drafts, nd, P, hist, lens)
        acc, best, com = oracle.accept_commit(drafts, nd, P, hist, lens)
        assert np.array_equal(acc, e_acc) and np.array_equal(best, e_best) and np.array_equal(com, e_com)
        assert np.array_equal(hist, e_hist) and np.array_equal(lens, e_lens)


def test_no_drafts_commits_the_plain_greedy_token():
    drafts = np.full((1, 2, 3), -1, np.int32)
    P = np.array([[[42, 1, 2, 3], [9, 9, 9, 9]]], np.int32)
    hist = np.full((1, 4), -1, np.int32)
    hist[0, 0] = 7
    lens = np.array([1], np.int32)
    acc, best, com = oracle.accept_commit(drafts, np.array([0], np.int32), P, hist, lens)
    assert acc.tolist() == [0] and best.tolist() == [0] and com[0].tolist() == [42, -1, -1, -1]
    assert hist[0].tolist() == [7, 42, -1, -1] and lens.tolist() == [2]


# ----------------------------------------------------------------------------- mixing (Section 4.3)
def brute_context_next_token(hist, q, w, topk):
    """Groups keyed by the next token only; the row comes from the latest occurrence."""
    hist = [int(t) for t in hist]
    L = len(hist)
    if L < q + w:
        return []
    groups = {}
    for i in range(L - q - w + 1):
        if hist[i:i + q] == hist[L - q:]:
            cnt, _ = groups.get(hist[i + q], (0, -1))
            groups[hist[i + q]] = (cnt + 1, i)
    order = sorted(groups.items(), key=lambda kv: (-kv[1][0], -kv[1][1]))[:topk]
    return [(tuple(hist[last + q:last + q + w]), cnt, last) for _, (cnt, last) in order]


def brute_mix(hist, qs, topk, B, w, flags, T):
    from test_oracle_context import brute_context, brute_context_partial
    rows, src, cnt = [], [], []
    ctx_cap = max(0, B - ((flags >> 8) & 0xFF))
    for q in qs:
        if flags & 8:       # occurrences near the end count too
            found = brute_context_partial(hist, q, w, topk, 1 if flags & 4 else w)
        else:
            found = brute_context(hist, q, w, topk) if not flags & 4 else brute_context_next_token(hist, q, w, topk)
        for c, n, _ in found:
            if len(rows) >= ctx_cap:
                break
            if (flags & 1) and list(c) in rows:
                continue
            rows.append(list(c)); src.append(q); cnt.append(n)
    if (flags & 2) and T is not None and len(hist) > 0:
        x = int(hist[-1])
        for r in range(T.shape[1]):
            if len(rows) == B:
                break
            chain, s = [], int(T[x, r])
            for _ in range(w):
                chain.append(s)
                s = int(T[s, 0])
            if (flags & 1) and chain in rows:
                continue
            rows.append(chain); src.append(0); cnt.append(0)
    return rows, src, cnt


def test_mixing_against_brute_force():
    g = np.random.default_rng(5)
    V, k_tab = 5, 3
    for trial in range(300):
        T = np.stack([g.permutation(V)[:k_tab] for _ in range(V)]).astype(np.int32)
        L = int(g.integers(0, 60))
        hist = g.integers(0, V, L).astype(np.int32)
        n_q = int(g.integers(0, 4))
        qs = [int(q) for q in g.permutation([1, 2, 3, 4])[:n_q]]
        topk, B, w = int(g.integers(1, 5)), int(g.integers(1, 9)), int(g.integers(1, 5))
        flags = int(g.integers(0, 16)) | (oracle.flag_reserve(int(g.integers(0, B + 2))) if trial % 3 == 0 else 0)
        cap = (L + 3) // 4 * 4 + 4
        h2 = np.full((1, cap), -1, np.int32)
        h2[0, :L] = hist
        drafts, nd, src, cnt = oracle.draft_batch(h2, np.array([L], np.int32), qs, topk, B, w, flags, T)
        rows, esrc, ecnt = brute_mix(hist, qs, topk, B, w, flags, T)
        n = len(rows)
        assert nd[0] == n
        assert drafts[0, :n].tolist() == rows and (drafts[0, n:] == -1).all()
        assert src[0, :n].tolist() == esrc and (src[0, n:] == -1).all()
        assert cnt[0, :n].tolist() == ecnt and (cnt[0, n:] == 0).all()


def test_context_rows_come_first_then_model_rows_in_rank_order():
    T = np.array([[1, 2, 0], [2, 0, 1], [0, 1, 2]], np.int32)   # top-1 chain 0->1->2->0
    hist = np.array([[0, 1, 2, 0, 1, 2, 0, -1]], np.int32)
    drafts, nd, src, cnt = oracle.draft_batch(hist, np.array([7], np.int32), [1], 2, 4, 2, 3, T)
    # context after token 0: (1,2) seen twice; model ranks: (1,2) duplicate dropped, (2,0), (0,1)
    assert nd[0] == 3 and drafts[0].tolist() == [[1, 2], [2, 0], [0, 1], [-1, -1]]
    assert src[0].tolist() == [1, 0, 0, -1] and cnt[0].tolist() == [2, 0, 0, 0]
    drafts, nd, src, _ = oracle.draft_batch(hist, np.array([7], np.int32), [1], 2, 4, 2, 2, T)  # no dedup
    assert nd[0] == 4 and drafts[0].tolist() == [[1, 2], [1, 2], [2, 0], [0, 1]]


def test_rows_reserved_for_the_model_cap_the_context_rows():
    T = np.array([[1, 2, 0], [2, 0, 1], [0, 1, 2]], np.int32)
    # after 0: (1,2) at 0, (2,1) at 3, (1,1) at 6, each once => ranked by recency: (1,1), (2,1), (1,2)
    hist = np.array([[0, 1, 2, 0, 2, 1, 0, 1, 1, 0, -1, -1]], np.int32)
    lens = np.array([10], np.int32)
    d, nd, src, _ = oracle.draft_batch(hist, lens, [1], 4, 4, 2, 3, T)
    assert nd[0] == 4 and src[0].tolist() == [1, 1, 1, 0]
    assert d[0].tolist() == [[1, 1], [2, 1], [1, 2], [2, 0]]      # model rank 0 = (1,2) is a duplicate, rank 1 = (2,0)
    d, nd, src, _ = oracle.draft_batch(hist, lens, [1], 4, 4, 2, 3 | oracle.flag_reserve(2), T)
    assert nd[0] == 4 and src[0].tolist() == [1, 1, 0, 0]
    # the context row (1,2) was cut by the reservation, so the model's (1,2) is not a duplicate of a row taken
    assert d[0].tolist() == [[1, 1], [2, 1], [1, 2], [2, 0]]
    d, nd, src, _ = oracle.draft_batch(hist, lens, [1], 4, 4, 2, 3 | oracle.flag_reserve(9), T)
    assert src[0, :nd[0]].tolist() == [0] * int(nd[0])                        # everything reserved: model rows only


def test_context_row_with_a_token_outside_the_vocabulary_is_passed_over():
    # after token 1: (2, 9) at 1 and (3, 1) at 4, once each => ranked by recency (3, 1), (2, 9); with V = 5 the
    # token 9 is not a vocabulary entry, so that row takes no draft row (and the rows behind it move up)
    T = np.array([[1, 2], [2, 0], [0, 1], [4, 0], [0, 3]], np.int32)
    hist = np.array([[1, 2, 9, 1, 3, 1, -1, -1]], np.int32)
    lens = np.array([6], np.int32)
    d, nd, src, cnt = oracle.draft_batch(hist, lens, [1], 4, 4, 2, 1, None)          # vocabulary unknown: both rows
    assert nd[0] == 2 and d[0, :2].tolist() == [[3, 1], [2, 9]]
    d, nd, src, cnt = oracle.draft_batch(hist, lens, [1], 4, 4, 2, 1, None, V=5)
    assert nd[0] == 1 and d[0].tolist() == [[3, 1], [-1, -1], [-1, -1], [-1, -1]] and src[0].tolist() == [1, -1, -1, -1]
    d, nd, src, cnt = oracle.draft_batch(hist, lens, [1], 4, 4, 2, 3, T)              # V from the table; model rows follow
    assert nd[0] == 3 and d[0, :3].tolist() == [[3, 1], [2, 0], [0, 1]] and src[0, :3].tolist() == [1, 0, 0]
    # brute force on random histories over {0..5} with V = 4: rows holding 4 or 5 vanish, the order of the rest is kept
    g = np.random.default_rng(17)
    for _ in range(100):
        L = int(g.integers(4, 50))
        h = g.integers(0, 6, L).astype(np.int32)
        h[-1] = g.integers(0, 4)
        w, topk = int(g.integers(1, 4)), int(g.integers(1, 6))
        h2 = np.full((1, (L + 3) // 4 * 4 + 4), -1, np.int32)
        h2[0, :L] = h
        rows, _, _ = brute_mix(h, [2, 1], topk, 64, w, 1, None)
        keep = [r for r in rows if all(0 <= t < 4 for t in r)]
        d, nd, _, _ = oracle.draft_batch(h2, np.array([L], np.int32), [2, 1], topk, 64, w, 1, None, V=4)
        assert d[0, :nd[0]].tolist() == keep


def test_ablation_counters_hand_example():
    # three sequences, B = 3, w = 2
    src = np.array([[1, 1, 0], [2, 0, -1], [0, 0, 0]], np.int32)
    acc = np.array([2, 0, -1], np.int32)          # accepted two tokens / nothing / could not commit
    best = np.array([1, 0, -1], np.int32)
    st = oracle.accumulate_stats(acc, best, src, w=2)
    assert st[:3].tolist() == [1, 0, 1]           # accepted lengths 0, 1, 2
    assert st[3:6].tolist() == [0, 1, 0]          # the accepted row was row 1
    assert st[6:11].tolist() == [0, 1, 0, 0, 0]   # ... which came from the q = 1 context strategy
    assert st[11:16].tolist() == [5, 2, 1, 0, 0]  # rows allocated: model 5, q=1 2, q=2 1
    st2 = oracle.accumulate_stats(acc, best, src, w=2, stats=st.copy())
    assert np.array_equal(st2, 2 * st)
