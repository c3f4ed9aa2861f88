"""Pins for the oracle's frequency-weighted continuation and suffix score (merged occurrences of the
longest match; draft limits and minimum token probability from the paper's drafting table)."""
import os

import numpy as np

from oracle import hvd_oracle as O
from tests.test_oracle_lookup import enumerate_matches, pack

f32 = np.float32


def brute_freq(h, K, l_max=64, min_match=2, min_prob=0.1, max_occ=256):
    """Independent restatement with Python containers: group the continuations of all occurrences."""
    h = list(h)
    n = len(h)
    pairs = enumerate_matches(h, l_max)
    if not pairs:
        return [], f32(0)
    L = max(l for _, l in pairs)
    if L < min_match:
        return [], f32(0)
    occ = sorted(e for e, l in pairs if l == L)
    limit = min(K, L)
    if len(occ) > max_occ:
        e = occ[-1]
        d = h[e:e + min(limit, n - e)]
        return d, f32(len(d))
    draft, score = [], f32(0)
    while len(draft) < limit:
        s = len(draft)
        groups = {}
        for e in occ:
            if e + s < n:
                groups.setdefault(h[e + s], []).append(e)
        if not groups:
            break
        tok = max(groups, key=lambda x: (len(groups[x]), max(groups[x])))
        prob = f32(len(groups[tok])) / f32(len(occ))
        if prob < f32(min_prob):
            break
        draft.append(tok)
        score = f32(score + prob)
        occ = groups[tok]
    return draft, score


def run_one(h, K, **kw):
    flat, off, cap, ln = pack([h])
    out = O.lookup_freq(flat, off, cap, ln, [K], k_cap=max(K, 1), **kw)
    return list(out.draft[0, :out.draft_len[0]]), out.score[0], out


def test_against_python_restatement():
    rng = np.random.default_rng(41)
    for _ in range(3000):
        n = int(rng.integers(0, 48))
        h = list(rng.integers(0, int(rng.integers(1, 4)), n))
        K = int(rng.integers(1, 8))
        kw = dict(l_max=int(rng.choice([2, 3, 64])), min_match=int(rng.choice([1, 2])),
                  min_prob=float(rng.choice([0.1, 0.34, 0.5])), max_occ=int(rng.choice([2, 5, 256])))
        d, sc, out = run_one(h, K, **kw)
        wd, wsc = brute_freq(h, K, **kw)
        assert d == wd and sc == wsc, (h, K, kw, d, sc, wd, wsc)
        assert (out.draft[0, len(d):] == -1).all()


def test_single_occurrence_is_the_plain_draft():
    rng = np.random.default_rng(42)
    h = list(rng.permutation(100000)[:500] + 5)
    h[-6:] = h[100:106]
    h[-7] = h[99] + 1
    d, sc, out = run_one(h, 4)
    flat, off, cap, ln = pack([h])
    plain = O.lookup(flat, off, cap, ln, [4], k_cap=4)
    assert d == list(plain.draft[0, :plain.draft_len[0]]) == h[106:110] and sc == 4.0 and out.match_cnt[0] == 1


def test_hand_worked_merge():
    # suffix "7 8" occurs four times before the end, followed by 1 2 / 1 3 / 4 5 / 1 3:
    # step 0: token 1 on 3 of 4 (prob 0.75); step 1 among those three: 3 on 2 of 3 (prob 2/3); the walk
    # then needs a third token, the two survivors continue with 9 and 6: tie 1:1 -> the later occurrence (6)
    # (different separators 50..53 keep the match at two tokens)
    h = [7, 8, 1, 2, 50, 7, 8, 1, 3, 9, 51, 7, 8, 4, 5, 52, 7, 8, 1, 3, 6, 53, 7, 8]
    d, sc, out = run_one(h, 3, spec_factor=0.0)
    assert out.match_len[0] == 2 and out.match_cnt[0] == 4
    assert d == [1, 3, 6]
    assert sc == f32(f32(f32(0.75) + f32(2) / f32(3)) + f32(0.5))
    # with the draft limited to the match length (factor 1.0) only two tokens come out
    d, sc, _ = run_one(h, 3)
    assert d == [1, 3] and sc == f32(f32(0.75) + f32(2) / f32(3))


def test_minimum_probability_cut():
    def fan(k):          # suffix "5 6" followed by k different tokens, one occurrence each
        h = []
        for i in range(k):
            h += [5, 6, 100 + i, 200 + i]
        return h + [5, 6]
    d, sc, _ = run_one(fan(11), 4)            # 1/11 < 0.1: nothing is drafted
    assert d == [] and sc == 0.0
    d, sc, _ = run_one(fan(10), 4)            # 1/10 == 0.1f: not below the minimum; the latest occurrence wins
    assert d == [109, 209] and sc == f32(f32(0.1) + f32(1.0))
    d, sc, _ = run_one(fan(12), 4, max_occ=8)    # more occurrences than are merged: the latest one alone
    assert d == [111, 211] and sc == 2.0


def test_freq_select_hand_cases():
    """Rule of the frequency-based hybrid baseline: cache draft iff non-empty and score >= threshold."""
    out = O.FreqOut(np.array([[5, 6, -1], [7, -1, -1], [-1, -1, -1], [8, 9, 4]], np.int32),
                    np.array([2, 1, 0, 3], np.int32), None, None, None,
                    np.array([1.5, 0.99, 0.0, 1.0], np.float32))
    md = np.array([[1, 2, 3], [1, 2, 3], [1, 2, 3], [1, 2, 3]], np.int32)
    ml = np.array([3, 2, 5, -1], np.int32)
    sel, sd, sl = O.freq_select(out, 1.0, md, ml)
    assert list(sel) == [1, 0, 0, 1]
    assert list(sl) == [2, 2, 3, 3]
    assert sd.tolist() == [[5, 6, -1], [1, 2, -1], [1, 2, 3], [8, 9, 4]]
    sel, sd, sl = O.freq_select(out, 0.0)               # no model draft: empty selection when not chosen
    assert list(sel) == [1, 1, 0, 1] and list(sl) == [2, 1, 0, 3]
    assert sd[2].tolist() == [-1, -1, -1]


def test_hand_worked_fixture():
    path = os.path.join(os.path.dirname(__file__), "golden", "frequency_walk_cases.txt")
    rows = [r for r in open(path) if r.strip() and not r.startswith("#")]
    assert len(rows) >= 7
    for r in rows:
        f = [x.strip() for x in r.rstrip("\n").split("|")]
        h = [int(x) for x in f[0].split()]
        K, sf, mp, mo, L, cnt = int(f[1]), float(f[2]), float(f[3]), int(f[4]), int(f[5]), int(f[6])
        want_d = [int(x) for x in f[7].split()]
        want_sc = f32(0)
        for t in f[8].split():
            a, b = t.split("/")
            want_sc = f32(want_sc + f32(a) / f32(b))
        d, sc, out = run_one(h, K, spec_factor=sf, min_prob=mp, max_occ=mo)
        assert (int(out.match_len[0]), int(out.match_cnt[0]), d, sc) == (L, cnt, want_d, want_sc), r
