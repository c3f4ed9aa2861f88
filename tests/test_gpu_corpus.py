"""GPU parity of the lookup over [shared warm-up corpus, own history] against the oracle, bit for bit."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from tests import gpu_helpers as G
from tests.test_oracle_lookup import pack

pytestmark = pytest.mark.gpu

NAMES = ("draft", "draft_len", "match_len", "match_pos", "match_src", "match_cnt")


class CorpusRunner:
    def __init__(self, max_batch, k_cap, max_hist_len, **cfg):
        import paper_2606_01019_b200 as H
        self.k_cap = k_cap
        self.ctx = H.Context(max_batch=max_batch, k_cap=k_cap, max_hist_len=max(max_hist_len, 1), max_rows=1,
                             max_vocab=1, **cfg)

    def set_corpus(self, corpus, pad_front=0):
        """Registers the corpus; pad_front (a multiple of 4 tokens) places it inside a larger allocation
        filled with a value that would match everything if it were read."""
        import torch
        if corpus is None:
            self.ctx.hvd_set_corpus(None)
            return
        buf = np.concatenate([np.zeros(pad_front, np.int32), np.asarray(corpus, np.int32), np.zeros(8, np.int32)])
        self.buf = torch.as_tensor(buf, device="cuda")
        self.ctx.hvd_set_corpus(self.buf[pad_front:pad_front + len(corpus)], len(corpus))

    def __call__(self, flat, off, cap, ln, K, n_max=None):
        import torch
        B = len(ln)
        dev = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a, dt), device="cuda")
        i32 = lambda *shape: torch.full(shape, -12345, dtype=torch.int32, device="cuda")
        out = dict(draft=i32(B, self.k_cap), draft_len=i32(B), match_len=i32(B), match_pos=i32(B), match_src=i32(B),
                   match_cnt=i32(B))
        self.ctx.hvd_lookup_corpus(B, dev(flat, np.int32), dev(off, np.int64), dev(cap, np.int32), dev(ln, np.int32),
                                   dev(K, np.int32), int(max(ln.max(), 0)) if n_max is None else n_max, out["draft"],
                                   out["draft_len"], out["match_len"], out["match_pos"], out["match_src"],
                                   out["match_cnt"])
        torch.cuda.synchronize()
        return {k: v.cpu().numpy() for k, v in out.items()}

    def close(self):
        self.ctx.close()


def check(got, want):
    for k in NAMES:
        G.assert_equal(k, got[k], getattr(want, k))


def with_separators(rng, corpus, k):
    corpus = np.array(corpus, np.int32)
    if len(corpus):
        corpus[rng.integers(0, len(corpus), k)] = -1 - rng.integers(0, 3, k)
    return corpus


@pytest.mark.parametrize("m", [0, 1, 2, 3, 5, 37, 8191, 8192, 8193, 8194, 30000])
def test_random_small_vocabularies(m):
    rng = np.random.default_rng(200 + m)
    B, k_cap = 70, int(rng.choice([4, 8, 33, 64]))
    vocab = int(rng.integers(2, 5))
    hs = [list(rng.integers(0, vocab, int(rng.integers(0, 300)))) for _ in range(B)]
    flat, off, cap, ln = pack(hs, extra_cap=int(rng.integers(0, 3)))
    K = rng.integers(0, k_cap + 1, B).astype(np.int32)
    cfg = dict(l_max=int(rng.choice([2, 3, 64])), min_match=int(rng.choice([1, 2, 3])), spec_factor=float(rng.choice([1.0, 4.0])))
    run = CorpusRunner(B, k_cap, int(cap.max()), **cfg)
    for rep in range(2):   # the second call finds the scratch as the first one left it
        corpus = with_separators(rng, rng.integers(0, vocab, m), int(rng.integers(0, 1 + m // 40)))
        run.set_corpus(corpus, pad_front=4 * rep)
        got = run(flat, off, cap, ln, K)
        want = O.lookup_corpus(flat, off, cap, ln, K, corpus, k_cap=k_cap, nthreads=8, **cfg)
        check(got, want)
    run.close()


def test_long_matches_in_a_large_vocabulary():
    """Spans of a document planted in the corpus and in the histories: long matches (up to l_max and
    beyond), both sources winning, ties between the sources, drafts cut at separators and at the end."""
    rng = np.random.default_rng(17)
    doc = rng.permutation(10**6)[:5000].astype(np.int32)
    pieces = []
    for _ in range(40):
        a = int(rng.integers(0, 4800)); pieces += [doc[a:a + int(rng.integers(5, 200))], np.array([-1], np.int32)]
        pieces.append(rng.integers(10**6, 2 * 10**6, int(rng.integers(0, 500))).astype(np.int32))
    corpus = np.concatenate(pieces)
    hs = []
    for b in range(96):
        own = rng.integers(2 * 10**6, 3 * 10**6, int(rng.integers(1, 600))).astype(np.int32)
        a = int(rng.integers(0, 4800)); span = doc[a:a + int(rng.integers(1, 120))]
        if b % 3 == 0:    # the history also holds the span earlier
            hs.append(np.concatenate([own, span, own[:7], span]))
        else:
            hs.append(np.concatenate([own, span]))
    flat, off, cap, ln = pack(hs, extra_cap=2)
    K = rng.integers(1, 65, len(hs)).astype(np.int32)
    run = CorpusRunner(len(hs), 64, int(cap.max()), spec_factor=2.0)
    run.set_corpus(corpus)
    got = run(flat, off, cap, ln, K)
    want = O.lookup_corpus(flat, off, cap, ln, K, corpus, k_cap=64, spec_factor=2.0, nthreads=8)
    check(got, want)
    assert (want.match_src == 1).sum() >= 10 and ((want.match_src == 0) & (want.match_len > 0)).sum() >= 10
    assert want.match_len.max() == 64 and (want.match_cnt >= 2).sum() >= 5
    # unregistering gives the plain lookup back
    run.set_corpus(None)
    got = run(flat, off, cap, ln, K)
    plain = O.lookup(flat, off, cap, ln, K, k_cap=64, spec_factor=2.0, nthreads=8)
    for k in ("draft", "draft_len", "match_len", "match_pos", "match_cnt"):
        G.assert_equal(k, got[k], getattr(plain, k))
    assert (got["match_src"] == 0).all()
    run.close()


@pytest.mark.parametrize("name,B,n", [("C5", 200, (64, 4096)), ("C3", 64, (256, 2048)), ("C2", 64, 16384)])
def test_workload_requests_and_warm_up_traces(name, B, n):
    w = W.CONFIGS[name].scaled(B=B, n=n)
    rq = W.make_requests(w)
    corpus = W.make_corpus(w, n_traces=24)
    run = CorpusRunner(rq.B, w.k_cap, int(rq.hist_cap.max()), l_max=w.l_max, min_match=w.min_match)
    run.set_corpus(corpus)
    got = run(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K)
    want = O.lookup_corpus(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, corpus, k_cap=w.k_cap, l_max=w.l_max,
                           min_match=w.min_match, nthreads=8)
    check(got, want)
    if name != "C2":
        assert (want.match_src == 1).sum() >= 3
    run.close()


@pytest.mark.parametrize("min_match,l_max", [(2, 64), (1, 64), (2, 1), (3, 5)])
def test_long_buckets(min_match, l_max):
    """Keys that occur thousands of times (runs of one token, a two-token cycle): every CTA of a request
    gets candidates, counts run into the thousands, and the longest lengths saturate at l_max."""
    rng = np.random.default_rng(31)
    corpus = np.concatenate([np.full(9000, 5, np.int32), [-1], np.tile(np.array([7, 8], np.int32), 4000), [-1],
                             rng.integers(0, 3, 6000).astype(np.int32), np.full(70, 5, np.int32), [9]])
    hs = [[5] * 10, [5] * 100, [1, 5], [7, 8] * 40, [8, 7, 8], [3, 7, 8, 7], list(rng.integers(0, 3, 50)), [9, 5, 5, 5],
          [5] * 3 + [6] + [5] * 3]
    flat, off, cap, ln = pack(hs)
    K = np.full(len(hs), 8, np.int32)
    cfg = dict(min_match=min_match, l_max=l_max, spec_factor=2.0)
    run = CorpusRunner(len(hs), 8, 128, **cfg)
    run.set_corpus(corpus)
    want = O.lookup_corpus(flat, off, cap, ln, K, corpus, k_cap=8, nthreads=8, **cfg)
    check(run(flat, off, cap, ln, K), want)
    if l_max >= min_match:
        assert want.match_cnt.max() > 3000
    else:
        assert (want.match_len == 0).all()
    run.close()


def test_degenerate_requests_and_bad_arguments():
    import torch
    import paper_2606_01019_b200 as H
    corpus = np.array([5, 5, 5, -1, 1, 2, 1, 2, 9, -1, 3, 4], np.int32)
    hs = [[], [5], [5, 5], [1, 2], [2, 1, 2], [9, 9, 9], [3, 4], [7, 3], list(range(50)), [-1, 1, 2]]
    flat, off, cap, ln = pack(hs)
    K = np.full(len(hs), 4, np.int32)
    run = CorpusRunner(len(hs), 4, 64, min_match=1)
    run.set_corpus(corpus)
    check(run(flat, off, cap, ln, K), O.lookup_corpus(flat, off, cap, ln, K, corpus, k_cap=4, min_match=1))
    bad = ln.copy(); bad[4] = -3; bad[8] = 10**6       # unusable lengths read as empty histories
    check(run(flat, off, cap, bad, K, n_max=64), O.lookup_corpus(flat, off, cap, bad, K, corpus, k_cap=4, min_match=1))
    buf = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(H.HvdError):
        run.ctx.hvd_set_corpus(buf[1:], 8)             # not 16-byte aligned
    run.close()
