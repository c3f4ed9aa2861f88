"""Pins for the oracle's prefix verification (Sec. 3.1 Verify read only as far as (a, z) depend on the logits)."""
import os

import numpy as np
import pytest

from oracle import hvd_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def one_request(draft, targets, k_cap, V=12, cap_extra=80, n0=5, select=1, poison=None):
    """Logits of one request with the strict maximum of row i at targets[i]; rows listed in `poison` hold NaN."""
    m = len(draft)
    rows = len(targets)
    logits = np.random.default_rng(1).normal(0, 1, (rows, V)).astype(np.float32)
    for i, t in enumerate(targets):
        logits[i, t] = 20.0
    for i in (poison or []):
        logits[i, :] = np.nan
    hist = np.full(n0 + cap_extra, -7, np.int32); hist[:n0] = np.arange(n0) + 40
    hist_len = np.array([n0], np.int32)
    state = np.zeros(1, O.STATE_DTYPE); state["sel_bits"] = 0b1011; state["acc_ring"] = 0x0102
    sd = np.full((1, k_cap), -1, np.int32); sd[0, :m] = draft
    kw = dict(k_cap=k_cap, hist=hist, hist_off=[0], hist_cap=[n0 + cap_extra], hist_len=hist_len, state=state)
    return logits, sd, [m], [select], kw


BIG = 1 << 30    # a batch so heavy that every boundary pays: two rows, two rows, then doubling
EVERY = dict(boundary_bytes=1)   # ... and the same windows for the small cases below


def test_windows_by_hand():
    assert O.prefix_windows(1, BIG) == [0, 2]
    assert O.prefix_windows(2, BIG) == [0, 3]
    assert O.prefix_windows(3, BIG) == [0, 2, 4]
    assert O.prefix_windows(4, BIG) == [0, 2, 5]
    assert O.prefix_windows(8, BIG) == [0, 2, 4, 9]
    assert O.prefix_windows(16, BIG) == [0, 2, 4, 8, 17]
    assert O.prefix_windows(32, BIG) == [0, 2, 4, 8, 16, 33]
    assert O.prefix_windows(64, BIG) == [0, 2, 4, 8, 16, 32, 65]
    # by size (worked by hand from the rule: first window >= 64 MiB, stop when rows left / 2^j < 128 MiB)
    MiB = 1 << 20
    assert O.prefix_windows(32, 256 * 151936 * 2) == [0, 2, 4, 8, 16, 33]     # 74.2 MiB per row index: 17 rows left / 16 = 79 MiB
    assert O.prefix_windows(16, 64 * 128256 * 2) == [0, 5, 17]                # 15.7 MiB: first window 5 rows, 12 left / 2 = 94 MiB
    assert O.prefix_windows(64, 32 * 128256 * 2) == [0, 9, 18, 65]            # 7.8 MiB: 9 rows, 56 left / 2 = 219, 47 left / 4 = 92
    assert O.prefix_windows(32, 512 * 128256 * 2) == [0, 2, 4, 8, 16, 33]     # 125 MiB
    assert O.prefix_windows(8, 4 * 32000 * 4) == [0, 9]                       # 0.5 MiB: one window, the plain verification
    assert O.prefix_windows(64, 64 * MiB) == [0, 2, 4, 8, 16, 32, 65]         # 49 rows left * 64 / 16 = 196 MiB: on; 33 * 64 / 32 = 66: stop
    assert O.prefix_windows(64, 1) == [0, 65]


def test_hand_worked_fixture_and_rows_read_by_hand():
    # the accepted-length fixture of the full verification: same a and z
    for line in open(os.path.join(GOLDEN, "accepted_length_cases.txt")):
        line = line.split("#")[0].rstrip("\n")
        if not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        draft = [int(x) for x in f[0].split()]; targets = [int(x) for x in f[1].split()]
        a = int(f[2]); z = [int(x) for x in f[3].split()]
        logits, sd, sl, sel, kw = one_request(draft, targets, k_cap=4, V=50)
        out = O.verify_commit_prefix(logits, O.F32, 50, np.array([0, len(targets)]), 0, sd, sl, sel, **kw, **EVERY)
        assert out.accepted[0] == a and list(out.committed[0, :a + 1]) == z and (out.committed[0, a + 1:] == -1).all(), line
        assert list(kw["hist"][5:5 + a + 1]) == z and kw["hist_len"][0] == 5 + a + 1
        assert kw["state"]["sel_bits"][0] == (0b1011 << 1 | 1) and kw["state"]["acc_ring"][0] == (0x0102 << 8 | a)
    # rows looked at, k_cap = 8: windows [0,2) [2,4) [4,9).  Draft 1..8; the target agrees up to position a.
    draft = [1, 2, 3, 4, 5, 6, 7, 8]
    by_hand = {0: 2, 1: 2, 2: 4, 3: 4, 4: 9, 5: 9, 6: 9, 7: 9, 8: 9}
    for a, want in by_hand.items():
        targets = draft[:a] + [0] + [9] * (8 - a)            # row a carries 0 (never a draft token)
        logits, sd, sl, sel, kw = one_request(draft, targets, k_cap=8)
        out = O.verify_commit_prefix(logits, O.F32, 12, np.array([0, 9]), 0, sd, sl, sel, **kw, **EVERY)
        assert out.accepted[0] == a and out.rows_read == want and out.rows_needed == a + 1, (a, out.rows_read)
    # a draft of 3 tokens, all accepted: rows 0..3, windows [0,2) and [2,4): 4 rows; of 2 tokens: 3 rows
    logits, sd, sl, sel, kw = one_request([1, 2, 3], [1, 2, 3, 7], k_cap=8)
    assert O.verify_commit_prefix(logits, O.F32, 12, np.array([0, 4]), 0, sd, sl, sel, **kw, **EVERY).rows_read == 4
    logits, sd, sl, sel, kw = one_request([1, 2], [1, 2, 7], k_cap=8)
    assert O.verify_commit_prefix(logits, O.F32, 12, np.array([0, 3]), 0, sd, sl, sel, **kw, **EVERY).rows_read == 3
    # an empty draft: one row
    logits, sd, sl, sel, kw = one_request([], [4], k_cap=8)
    out = O.verify_commit_prefix(logits, O.F32, 12, np.array([0, 1]), 0, sd, sl, sel, **kw, **EVERY)
    assert out.rows_read == 1 and out.accepted[0] == 0 and out.committed[0, 0] == 4


@pytest.mark.parametrize("k_cap", [1, 2, 3, 5, 8, 16, 33, 64])
def test_no_row_behind_the_stopping_window_is_looked_at(k_cap):
    """Every (draft length m, accepted length a): the rows behind the window in which the walk stops hold NaN,
    and the result is still that of the full verification of the clean logits; the rows looked at stay within
    twice the rows needed plus two."""
    edges = O.prefix_windows(k_cap, 12 * 4, 1)
    rng = np.random.default_rng(k_cap)
    for m in range(0, k_cap + 1):
        for a in sorted(set([0, 1, 2, 3, m // 2, m - 1, m]) & set(range(0, m + 1))):
            draft = [int(x) for x in rng.integers(1, 6, m)]
            targets = draft[:a] + [0] + [int(x) for x in rng.integers(1, 6, m - a)]   # row a rejects (or ends the draft)
            stop_hi = next(hi for hi in edges[1:] if a < hi)
            poison = list(range(min(stop_hi, m + 1), m + 1))
            logits, sd, sl, sel, kw = one_request(draft, targets, k_cap=k_cap, poison=poison)
            clean, sd2, sl2, sel2, kw2 = one_request(draft, targets, k_cap=k_cap)
            got = O.verify_commit_prefix(logits, O.F32, 12, np.array([0, m + 1]), 0, sd, sl, sel, **kw, **EVERY)
            want = O.verify_commit(clean, O.F32, 12, np.array([0, m + 1], np.int64), 0, sd2, sl2, sel2, **kw2)
            assert got.accepted[0] == want.accepted[0] == a
            assert (got.committed == want.committed).all() and got.n_commit[0] == want.n_commit[0]
            assert (kw["hist"] == kw2["hist"]).all() and kw["hist_len"][0] == kw2["hist_len"][0]
            assert kw["state"][0] == kw2["state"][0]
            assert got.rows_read == min(stop_hi, m + 1) and a + 1 <= got.rows_read <= 2 * (a + 1) + 2


def test_equals_the_full_verification_on_random_batches():
    rng = np.random.default_rng(5)
    for it in range(150):
        B = int(rng.integers(1, 9)); k_cap = int(rng.choice([1, 2, 4, 7, 16, 40, 64])); V = int(rng.choice([1, 2, 5, 30]))
        dtype = int(rng.choice([O.F32, O.BF16]))
        K = rng.integers(0, k_cap + 1, B)
        row_off = np.zeros(B + 1, np.int64); row_off[1:] = np.cumsum(K + 1)
        x = rng.integers(-3, 4, (int(row_off[-1]), V)).astype(np.float32)        # small integers: ties are common
        logits = x if dtype == O.F32 else (x.view(np.uint32) >> 16).astype(np.uint16)
        sel_len = np.minimum(rng.integers(-1, k_cap + 2, B), 70).astype(np.int32)
        sd = rng.integers(-1, V + 1, (B, k_cap)).astype(np.int32)
        # make some drafts agree with the target for a while
        for b in range(B):
            for i in range(int(rng.integers(0, k_cap + 1))):
                if i <= K[b]:
                    sd[b, i] = O.argmax_row(logits[row_off[b] + i], dtype) if i < K[b] + 1 else sd[b, i]
        n = rng.integers(0, 30, B).astype(np.int32)
        cap = (n + rng.integers(0, 2 * k_cap + 3, B)).astype(np.int32)
        if rng.random() < 0.3:
            n[int(rng.integers(0, B))] = int(rng.choice([-1, 1000]))
        hist_off = np.zeros(B, np.int64); hist_off[1:] = np.cumsum(cap[:-1])
        hist = rng.integers(0, 9, int(cap.sum()) + 1).astype(np.int32)
        state = np.zeros(B, O.STATE_DTYPE)
        state["sel_bits"] = rng.integers(0, 2**32, B, dtype=np.uint64).astype(np.uint32)
        state["acc_ring"] = rng.integers(0, 2**63, B, dtype=np.uint64) * 2 + 1
        select = rng.integers(0, 2, B).astype(np.int32)
        h1, l1, s1 = hist.copy(), n.copy(), state.copy()
        h2, l2, s2 = hist.copy(), n.copy(), state.copy()
        want = O.verify_commit(logits, dtype, V, row_off, 0, sd, sel_len, select, k_cap=k_cap, hist=h1, hist_off=hist_off,
                               hist_cap=cap, hist_len=l1, state=s1)
        bb = int(rng.choice([1, 1, 40, 64 << 20]))
        w0 = O.prefix_windows(k_cap, B * V * (4 if dtype == O.F32 else 2), bb)[1]
        got = O.verify_commit_prefix(logits, dtype, V, row_off, 0, sd, sel_len, select, k_cap=k_cap, hist=h2,
                                     hist_off=hist_off, hist_cap=cap, hist_len=l2, state=s2,
                                     boundary_bytes=bb)
        for k in ("accepted", "committed", "n_commit", "status"):
            assert (getattr(got, k) == getattr(want, k)).all(), (it, k)
        assert (h1 == h2).all() and (l1 == l2).all() and (s1 == s2).all(), it
        valid = want.status != O.REQ_BAD_LEN
        assert got.rows_needed == int((want.accepted[valid] + 1).sum())
        assert got.rows_needed <= got.rows_read <= 2 * got.rows_needed + w0 * int(valid.sum())   # twice the need plus the first window
