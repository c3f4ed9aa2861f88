"""Pins for the oracle's trace-replay labels (Sec. 3.3 label equation; App. B "Payoff Label Construction")."""
import numpy as np

from oracle import hvd_oracle as O
from tests.test_oracle_lookup import expected_from_pairs


def brute_labels(x, K, l_max=64, min_match=2):
    """For every prefix length t: draft from the pair enumerator, label straight from the equation
    y_t = max{l in 0..|d| : d[0:l] == x[t:t+l]}."""
    x = list(x)
    n = len(x)
    out = []
    for t in range(1, n + 1):
        L, e, c, d = expected_from_pairs(x[:t], K, l_max, min_match)
        y = max(l for l in range(len(d) + 1) if d[:l] == x[t:t + l])
        out.append((y, len(d), L, e, c))
    return out


def test_labels_against_the_equation_on_small_strings():
    rng = np.random.default_rng(21)
    for _ in range(300):
        n = int(rng.integers(1, 60))
        x = rng.integers(0, int(rng.integers(1, 5)), n)
        K = int(rng.integers(1, 9))
        got = O.replay_labels(x, K, k_cap=8)
        want = brute_labels(x, K)
        for j, (y, d, L, e, c) in enumerate(want):
            assert (got.label[j], got.draft_len[j], got.match_len[j], got.match_pos[j], got.match_cnt[j]) == (y, d, L, e, c), (list(x), K, j)


def test_hand_worked_trace():
    # trace 1 2 3 9 1 2 3 9 5: at t = 7 (prefix 1 2 3 9 1 2 3) the draft is 9 1 2 (match of length 3 at e = 3),
    # the continuation is 9 5: y = 1.  At t = 8 (prefix ... 3 9) the match is 1 2 3 9 (e = 4), draft 1 2 3 9,
    # continuation 5: y = 0.  At t = 6 the match "1 2" (e = 2) gives draft 3 9, continuation 3 9 5: y = 2.
    x = [1, 2, 3, 9, 1, 2, 3, 9, 5]
    out = O.replay_labels(x, 4, k_cap=4)
    assert (out.match_len[6], out.match_pos[6], out.draft_len[6], out.label[6]) == (3, 3, 3, 1)
    assert (out.match_len[7], out.match_pos[7], out.draft_len[7], out.label[7]) == (4, 4, 4, 0)
    assert (out.match_len[5], out.match_pos[5], out.draft_len[5], out.label[5]) == (2, 2, 2, 2)
    assert out.label[8] == 0 and (out.label[:5] == 0).all()          # nothing to match early, nothing follows the end


def test_repeated_document_is_fully_predictable():
    """x = D || D with all-distinct D: inside the second copy every draft continues the first copy, so the
    whole draft agrees with the trace (clipped by the end of the trace)."""
    rng = np.random.default_rng(22)
    m, K = 200, 8
    D = rng.permutation(10**6)[:m].astype(np.int32) + 1
    x = np.concatenate([D, D])
    out = O.replay_labels(x, K, k_cap=K)
    assert (out.label[:m + 1] == 0).all() and (out.match_len[:m + 1] == 0).all()
    for t in range(m + 2, 2 * m + 1):
        L = min(t - m, 64)
        d = min(K, L)
        assert out.match_len[t - 1] == L and out.match_pos[t - 1] == t - m and out.draft_len[t - 1] == d
        assert out.label[t - 1] == min(d, 2 * m - t)


def test_invariants_on_a_workload_history():
    import hvd_workloads as W
    rq = W.make_requests(W.CONFIGS["C2"].scaled(B=2, n=3000))
    x = rq.history(0)
    out = O.replay_labels(x, 16, k_cap=16, nthreads=4)
    assert ((0 <= out.label) & (out.label <= out.draft_len) & (out.draft_len <= np.minimum(16, out.match_len))).all()
    assert out.label.max() >= 4                      # the template copies do get replayed
    t = int(np.argmax(out.label)) + 1
    e, y = int(out.match_pos[t - 1]), int(out.label[t - 1])
    assert (x[e:e + y] == x[t:t + y]).all()
