"""Pins for the oracle's lookup over [shared warm-up corpus, own history] (Algorithm 1's cache
initialisation with the lookup rule of Sec. 3.2): slice-equality brute force, hand-worked cases,
reductions to the plain lookup, separator rules."""
import os

import numpy as np

from oracle import hvd_oracle as O
from tests.test_oracle_lookup import enumerate_matches, pack

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def brute_corpus(h, corpus, K, l_max=64, min_match=2):
    """Every (source, e, l) by slice equality; then the selection rules, written independently."""
    h, corpus = list(h), list(corpus)
    n, m = len(h), len(corpus)
    cands = [(l, 0, e) for e, l in enumerate_matches(h, l_max)]
    for e in range(1, m):
        if corpus[e] < 0:
            continue
        for l in range(1, min(l_max, e, n) + 1):
            seg = corpus[e - l:e]
            if min(seg) >= 0 and seg == h[n - l:n]:
                cands.append((l, 1, e))
    if not cands:
        return 0, 0, -1, 0, []
    # per (source, e) the longest length
    longest = {}
    for l, src, e in cands:
        longest[(src, e)] = max(longest.get((src, e), 0), l)
    L = max(longest.values())
    if L < min_match:
        return 0, 0, -1, 0, []
    at_L = [(src, e) for (src, e), l in longest.items() if l == L]
    hist_e = [e for src, e in at_L if src == 0]
    src, e = (0, max(hist_e)) if hist_e else (1, max(e for _, e in at_L))
    limit = min(K, L)
    if src == 0:
        draft = h[e:e + limit]
    else:
        draft = []
        for x in corpus[e:e + limit]:
            if x < 0:
                break
            draft.append(x)
    return L, src, e, len(at_L), draft


def run_one(h, corpus, K, **kw):
    flat, off, cap, ln = pack([h])
    out = O.lookup_corpus(flat, off, cap, ln, [K], corpus, k_cap=max(K, 1), **kw)
    return (int(out.match_len[0]), int(out.match_src[0]), int(out.match_pos[0]), int(out.match_cnt[0]),
            [int(x) for x in out.draft[0, :out.draft_len[0]]])


def test_against_slice_equality_brute_force():
    rng = np.random.default_rng(77)
    seen_src = set()
    for _ in range(4000):
        vocab = int(rng.integers(1, 4))
        h = list(rng.integers(0, vocab, int(rng.integers(0, 24))))
        corpus = list(rng.integers(0, vocab, int(rng.integers(0, 40))))
        for p in rng.integers(0, max(len(corpus), 1), int(rng.integers(0, 4))):   # separators
            if corpus:
                corpus[int(p)] = -1 - int(rng.integers(0, 3))
        K = int(rng.integers(1, 7))
        kw = dict(l_max=int(rng.choice([1, 2, 3, 64])), min_match=int(rng.choice([1, 2, 3])))
        got = run_one(h, corpus, K, **kw)
        want = brute_corpus(h, corpus, K, **kw)
        assert got == want, (h, corpus, K, kw, got, want)
        seen_src.add((got[0] > 0, got[1]))
    assert seen_src == {(False, 0), (True, 0), (True, 1)}


def test_hand_worked_fixture():
    rows = [r for r in open(os.path.join(GOLDEN, "corpus_match_cases.txt")) if r.strip() and not r.startswith("#")]
    assert len(rows) >= 9
    for r in rows:
        f = [x.strip() for x in r.split("|")]
        corpus, h = [int(x) for x in f[0].split()], [int(x) for x in f[1].split()]
        K, l_max, min_match, L, src, pos, cnt = (int(x) for x in f[2:9])
        draft = [int(x) for x in f[9].split()]
        assert run_one(h, corpus, K, l_max=l_max, min_match=min_match) == (L, src, pos, cnt, draft), r


def test_empty_corpus_is_the_plain_lookup():
    rng = np.random.default_rng(3)
    hs = [list(rng.integers(0, 3, int(rng.integers(0, 60)))) for _ in range(200)]
    flat, off, cap, ln = pack(hs)
    K = rng.integers(0, 9, len(hs)).astype(np.int32)
    a = O.lookup(flat, off, cap, ln, K, k_cap=8)
    b = O.lookup_corpus(flat, off, cap, ln, K, np.zeros(0, np.int32), k_cap=8)
    for k in ("draft", "draft_len", "match_len", "match_pos", "match_cnt"):
        assert (getattr(a, k) == getattr(b, k)).all(), k
    assert (b.match_src == 0).all()


def test_concatenation_reduces_to_the_plain_lookup():
    """One warm-up trace without separators: wherever the winning occurrence and its draft lie strictly
    inside the corpus, the plain lookup on corpus + [separator] + history finds the same match (shifted),
    because the plain rule also prefers the latest position, which puts the history first."""
    rng = np.random.default_rng(5)
    checked = 0
    for _ in range(3000):
        vocab = int(rng.integers(2, 5))
        h = list(rng.integers(0, vocab, int(rng.integers(1, 20))))
        corpus = list(rng.integers(0, vocab, int(rng.integers(2, 40))))
        K = int(rng.integers(1, 6))
        L, src, pos, cnt, draft = run_one(h, corpus, K)
        X = corpus + [-1] + h
        flat, off, cap, ln = pack([X])
        p = O.lookup(flat, off, cap, ln, [K], k_cap=K)
        m = len(corpus)
        lt = 0                                                     # common suffix of the corpus and the history
        while lt < min(m, len(h)) and corpus[m - 1 - lt] == h[len(h) - 1 - lt]:
            lt += 1
        if lt >= max(L, 1):
            continue       # an occurrence ending at the corpus end: the plain rule counts it, ours has no continuation for it
        assert int(p.match_len[0]) == L and int(p.match_cnt[0]) == cnt
        if L:
            assert int(p.match_pos[0]) == (pos if src else pos + m + 1)
            if src == 0 or pos + min(K, L) <= m:
                assert [int(x) for x in p.draft[0, :p.draft_len[0]]] == draft
                checked += 1
    assert checked > 500


def test_separator_rules():
    # a match may not contain a separator, nor extend across one
    assert run_one([1, 2, 3], [1, -1, 2, 3, 9], 4)[:4] == (2, 1, 4, 1)
    assert run_one([1, 2, 3], [1, 2, -5, 3, 9], 4, min_match=1)[:4] == (1, 1, 4, 1)
    # an occurrence whose continuation is a separator or the corpus end is not a candidate
    assert run_one([1, 2, 3], [1, 2, 3, -1, 1, 2, 3], 4)[0] == 0
    # the draft stops before a separator and at the corpus end
    assert run_one([7, 1, 2, 3], [1, 2, 3, 4, 5, -1, 6], 8, spec_factor=3.0)[4] == [4, 5]
    assert run_one([7, 1, 2, 3], [1, 2, 3, 4, 5], 8, spec_factor=3.0)[4] == [4, 5]
    # history tokens that happen to be negative never match a separator
    assert run_one([-1, 2], [5, -1, 2, 8], 4, min_match=1)[:4] == (1, 1, 3, 1)
    # the corpus cannot supply more context than the history has (l <= n)
    assert run_one([2], [1, 2, 3], 4, min_match=1)[:4] == (1, 1, 2, 1)


def test_sources_and_counts_on_planted_copies():
    rng = np.random.default_rng(9)
    doc = list(rng.permutation(10**5)[:300])
    corpus = doc[:100] + [-1] + doc[100:200] + [-1] + doc[50:150]
    # suffix from the second trace; it also occurs in the third trace (overlap 100..150)
    h = list(rng.permutation(10**5)[:40] + 10**6) + doc[110:130]
    L, src, pos, cnt, draft = run_one(h, corpus, 8)
    assert (L, src, cnt) == (20, 1, 2)
    assert pos == 202 + (130 - 50) and draft == doc[130:138]      # the latest corpus position wins
    # once the history itself holds the span twice, the history wins at equal length
    h2 = h + [5] + doc[110:130]
    L, src, pos, cnt, draft = run_one(h2, corpus, 8)
    assert (L, src, cnt) == (20, 0, 3) and pos == 60 and draft == [5] + doc[110:117]
