"""Pins for the oracle's suffix-match lookup (Sec. 3.2): brute-force enumeration on tiny inputs,
hand-worked fixtures, constructed cases, a library special case and invariants."""
import itertools
import os

import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from oracle import pipeline as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def pack(histories, extra_cap=0):
    """Flat array + offsets for a list of token lists."""
    off, cap, ln, parts, p = [], [], [], [], 0
    for h in histories:
        off.append(p); cap.append(len(h) + extra_cap); ln.append(len(h))
        parts.append(np.asarray(h, np.int32)); parts.append(np.full(extra_cap, -7, np.int32))
        p += len(h) + extra_cap
    flat = np.concatenate(parts) if parts else np.zeros(0, np.int32)
    if flat.size == 0:
        flat = np.zeros(1, np.int32)
    return flat, np.asarray(off, np.int64), np.asarray(cap, np.int32), np.asarray(ln, np.int32)


def enumerate_matches(h, l_max):
    """Every (e, l) with h[e-l:e] == h[n-l:n], 1 <= l <= min(l_max, e), 1 <= e <= n-1, listed the
    dumb way: slice equality for every pair, no incremental extension."""
    n = len(h)
    pairs = []
    for e in range(1, n):
        for l in range(1, min(l_max, e) + 1):
            if list(h[e - l:e]) == list(h[n - l:n]):
                pairs.append((e, l))
    return pairs


def expected_from_pairs(h, K, l_max, min_match):
    pairs = enumerate_matches(h, l_max)
    n = len(h)
    if not pairs:
        return 0, -1, 0, []
    L = max(l for _, l in pairs)
    if L < min_match:
        return 0, -1, 0, []
    es = sorted(e for e, l in pairs if l == L)
    e = es[-1]
    d = min(K, L, n - e)
    return L, e, len(es), list(h[e:e + d])


def check_batch(histories, K, l_max, min_match):
    flat, off, cap, ln = pack(histories)
    k_cap = max(K, 1)
    out = O.lookup(flat, off, cap, ln, np.full(len(histories), K, np.int32), k_cap=k_cap, l_max=l_max,
                   min_match=min_match)
    for b, h in enumerate(histories):
        L, e, c, d = expected_from_pairs(h, K, l_max, min_match)
        got = (int(out.match_len[b]), int(out.match_pos[b]), int(out.match_cnt[b]),
               list(out.draft[b, :out.draft_len[b]]))
        assert got == (L, e, c, d), (h, K, l_max, min_match, got, (L, e, c, d))
        assert (out.draft[b, out.draft_len[b]:] == -1).all()


def test_exhaustive_ternary_strings():
    hs = [list(t) for n in range(0, 9) for t in itertools.product(range(3), repeat=n)]
    check_batch(hs, K=4, l_max=64, min_match=2)
    check_batch(hs, K=2, l_max=3, min_match=1)


def test_exhaustive_binary_strings_len_10_to_12():
    hs = [list(t) for n in (10, 11, 12) for t in itertools.product(range(2), repeat=n)]
    check_batch(hs, K=5, l_max=4, min_match=2)
    check_batch(hs[::3], K=3, l_max=64, min_match=3)


def test_random_small_vocab_strings():
    rng = np.random.default_rng(1234)
    hs = [list(rng.integers(0, rng.integers(1, 5), rng.integers(0, 33))) for _ in range(10000)]
    check_batch(hs, K=6, l_max=64, min_match=2)
    check_batch(hs[:3000], K=1, l_max=5, min_match=1)


def test_hand_worked_fixture():
    for line in open(os.path.join(GOLDEN, "suffix_match_cases.txt")):
        line = line.split("#")[0].rstrip("\n")
        if not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        h = [int(x) for x in f[0].split()]
        K, l_max, mm, L, pos, cnt = (int(x) for x in f[1:7])
        draft = [int(x) for x in f[7].split()]
        flat, off, cap, ln = pack([h])
        out = O.lookup(flat, off, cap, ln, [K], k_cap=8, l_max=l_max, min_match=mm)
        assert (int(out.match_len[0]), int(out.match_pos[0]), int(out.match_cnt[0])) == (L, pos, cnt), line
        assert list(out.draft[0, :out.draft_len[0]]) == draft, line


def test_paper_constants_are_the_defaults():
    vals = {}
    for line in open(os.path.join(GOLDEN, "paper_constants.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            vals[line[0]] = line[1]
    import inspect
    sig = inspect.signature(O.lookup).parameters
    assert sig["l_max"].default == int(vals["suffix_cache_max_depth"])
    assert sig["spec_factor"].default == float(vals["max_spec_factor"])
    assert sig["spec_offset"].default == float(vals["max_spec_offset"])
    for c in W.CONFIGS.values():
        assert c.l_max == int(vals["suffix_cache_max_depth"])
        assert c.k_cap <= int(vals["suffix_cache_max_draft"])
    assert W.CONFIGS["C3"].b2 == float(vals["select_threshold"])


@pytest.mark.parametrize("T", [1, 2, 3, 63, 64, 65, 96])
def test_planted_tail(T):
    """i.i.d. history over a huge vocabulary, tail = copy of an earlier span preceded by a forced
    mismatch: the match is that span, its length min(T, 64), once."""
    rng = np.random.default_rng(T)
    n, V, K = 4000, 2**30, 16
    h = rng.permutation(V // 1024)[:n].astype(np.int32) * 7 + 3      # all tokens distinct
    e0 = 1700
    h[n - T:n] = h[e0 - T:e0]
    h[n - T - 1] = h[e0 - T - 1] + 1                                 # forced mismatch before the copy
    flat, off, cap, ln = pack([h])
    out = O.lookup(flat, off, cap, ln, [K], k_cap=K)
    if T < 2:
        assert out.match_len[0] == 0 and out.match_pos[0] == -1 and out.draft_len[0] == 0
        return
    L = min(T, 64)
    assert (out.match_len[0], out.match_pos[0], out.match_cnt[0]) == (L, e0, 1)
    d = min(K, L)
    assert out.draft_len[0] == d and (out.draft[0, :d] == h[e0:e0 + d]).all()


def test_repeated_span_count_and_latest():
    rng = np.random.default_rng(7)
    n, T, r = 3000, 10, 5
    h = (rng.permutation(1 << 20)[:n].astype(np.int32)) + 10
    span = h[100:100 + T].copy()
    ends = [100 + T]
    for j in range(1, r):
        s = 300 + 400 * j
        h[s:s + T] = span
        ends.append(s + T)
    h[n - T:n] = span
    flat, off, cap, ln = pack([h])
    out = O.lookup(flat, off, cap, ln, [8], k_cap=8)
    assert (out.match_len[0], out.match_cnt[0], out.match_pos[0]) == (T, r, ends[-1])
    assert (out.draft[0, :8] == h[ends[-1]:ends[-1] + 8]).all()


def test_all_equal_history():
    n = 300
    flat, off, cap, ln = pack([[9] * n])
    out = O.lookup(flat, off, cap, ln, [8], k_cap=8)
    # every e >= 64 matches with the capped length 64; e* = n-1 leaves one token to draft
    assert (out.match_len[0], out.match_pos[0], out.match_cnt[0], out.draft_len[0]) == (64, n - 1, n - 64, 1)


def test_special_case_equals_bytes_rfind():
    """With no depth cap the result is the longest proper suffix that also occurs earlier, which
    Python's bytes.rfind finds directly."""
    rng = np.random.default_rng(99)
    for _ in range(300):
        n = int(rng.integers(2, 200))
        h = rng.integers(0, int(rng.integers(1, 6)), n).astype(np.int32)
        s = bytes(h.astype(np.uint8))
        L = e = 0
        for l in range(n - 1, 0, -1):
            pos = s.rfind(s[n - l:], 0, n - 1)      # occurrence must end at or before n-1
            if pos >= 0:
                L, e = l, pos + l
                break
        cnt = 0
        if L:
            start = 0
            while True:
                pos = s.find(s[n - L:], start, n - 1)
                if pos < 0:
                    break
                cnt += 1
                start = pos + 1
        flat, off, cap, ln = pack([h])
        out = O.lookup(flat, off, cap, ln, [4], k_cap=4, l_max=1 << 20, min_match=1)
        if L == 0:
            assert out.match_len[0] == 0
        else:
            assert (out.match_len[0], out.match_pos[0], out.match_cnt[0]) == (L, e, cnt), h


def test_spec_factor_and_offset():
    h = [1, 2, 3, 4, 5, 6, 7, 8, 1, 2, 3, 4]         # suffix 1 2 3 4 matched at e = 4
    flat, off, cap, ln = pack([h])
    for factor, offset, want in [(1.0, 0.0, 4), (0.5, 0.0, 2), (0.5, 1.0, 3), (2.0, 0.0, 6),
                                 (0.0, 0.0, 6), (0.25, 0.5, 1), (0.1, 0.0, 0)]:
        out = O.lookup(flat, off, cap, ln, [6], k_cap=6, spec_factor=factor, spec_offset=offset)
        assert out.match_len[0] == 4 and out.match_pos[0] == 4
        assert out.draft_len[0] == want, (factor, offset)
        assert list(out.draft[0, :want]) == h[4:4 + want]


def test_invalid_lengths_and_k_are_neutral():
    flat, off, cap, ln = pack([[1, 2, 1, 2, 1, 2], [1, 2, 1, 2, 1, 2], [3, 3, 3, 3]], extra_cap=2)
    ln2 = np.array([-1, 99, 4], np.int32)
    out = O.lookup(flat, off, cap, ln2, [4, 4, 0], k_cap=4)
    assert list(out.match_len) == [0, 0, 3] and list(out.draft_len) == [0, 0, 0]
    assert (out.draft == -1).all()


@pytest.mark.parametrize("name", ["C1", "C2", "C5"])
def test_invariants_on_workloads(name):
    w = W.CONFIGS[name]
    if name == "C5":
        w = w.scaled(B=48, n=(64, 4096))
    rq = W.make_requests(w)
    lk = P.lookup(w, rq, nthreads=4)
    matched = 0
    for b in range(rq.B):
        h = rq.history(b)
        n, L, e, c, d = len(h), int(lk.match_len[b]), int(lk.match_pos[b]), int(lk.match_cnt[b]), int(lk.draft_len[b])
        assert (c >= 1) == (L >= w.min_match)
        if L == 0:
            assert e == -1 and d == 0
            continue
        matched += 1
        assert 1 <= e <= n - 1 and L <= min(64, e)
        assert (h[e - L:e] == h[n - L:n]).all()
        assert L == 64 or e == L or h[e - L - 1] != h[n - L - 1]        # maximal
        assert d == min(int(rq.K[b]), L, n - e) and (lk.draft[b, :d] == h[e:e + d]).all()
        # no later position matches as long, none anywhere matches longer (vectorised re-check)
        tail = h[n - L:n]
        win = np.lib.stride_tricks.sliding_window_view(h[:n - 1], L)     # windows ending at e = i + L
        hits = np.nonzero((win == tail).all(axis=1))[0] + L
        assert hits.max() == e and len(hits) == c
        if L < 64 and n - 1 > L:
            tail1 = h[n - L - 1:n]
            win1 = np.lib.stride_tricks.sliding_window_view(h[:n - 1], L + 1)
            assert not (win1 == tail1).all(axis=1).any()
    assert matched > 0
