"""GPU parity of the frequency-weighted cache draft, its score and the score-threshold selection
against the oracle: every output bit for bit (the probabilities are single IEEE divisions and the
score is an fp32 sum in step order on both sides)."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from tests import gpu_helpers as G
from tests.test_oracle_lookup import pack

pytestmark = pytest.mark.gpu

NAMES = ("draft", "draft_len", "match_len", "match_pos", "match_cnt")


class FreqRunner:
    def __init__(self, max_batch, k_cap, max_hist_len, **cfg):
        import paper_2606_01019_b200 as H
        self.k_cap = k_cap
        self.ctx = H.Context(max_batch=max_batch, k_cap=k_cap, max_hist_len=max(max_hist_len, 1), max_rows=1,
                             max_vocab=1, **cfg)

    def __call__(self, flat, off, cap, ln, K, min_prob, max_occ, threshold=None, model_draft=None, model_len=None,
                 n_max=None):
        import torch
        B = len(ln)
        dev = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a, dt), device="cuda")
        i32 = lambda *shape: torch.full(shape, -12345, dtype=torch.int32, device="cuda")
        out = dict(draft=i32(B, self.k_cap), draft_len=i32(B), score=torch.full((B,), -7.0, device="cuda"),
                   match_len=i32(B), match_pos=i32(B), match_cnt=i32(B))
        sel = dict(select=i32(B), sel_draft=i32(B, self.k_cap), sel_len=i32(B)) if threshold is not None else {}
        md = None if model_draft is None else dev(model_draft, np.int32)
        ml = None if model_len is None else dev(model_len, np.int32)
        self.ctx.hvd_lookup_freq(B, dev(flat, np.int32), dev(off, np.int64), dev(cap, np.int32), dev(ln, np.int32),
                                 dev(K, np.int32), int(max(ln.max(), 0)) if n_max is None else n_max, float(min_prob), int(max_occ),
                                 float(threshold if threshold is not None else 0.0), md, ml, out["draft"],
                                 out["draft_len"], out["score"], out["match_len"], out["match_pos"],
                                 out["match_cnt"], sel.get("select"), sel.get("sel_draft"), sel.get("sel_len"))
        torch.cuda.synchronize()
        return {k: v.cpu().numpy() for k, v in {**out, **sel}.items()}

    def close(self):
        self.ctx.close()


def check(got, want):
    for k in NAMES:
        G.assert_equal(k, got[k], getattr(want, k))
    G.assert_equal("score bits", got["score"].view(np.uint32), want.score.view(np.uint32))


@pytest.mark.parametrize("seed", range(6))
def test_random_small_vocabularies(seed):
    rng = np.random.default_rng(100 + seed)
    B, k_cap = 96, int(rng.choice([4, 8, 33, 64]))
    hs = [list(rng.integers(0, int(rng.integers(1, 5)), int(rng.integers(0, 400)))) for _ in range(B)]
    flat, off, cap, ln = pack(hs, extra_cap=int(rng.integers(0, 3)))
    K = rng.integers(0, k_cap + 1, B).astype(np.int32)
    cfg = dict(l_max=int(rng.choice([2, 3, 64])), min_match=int(rng.choice([1, 2])))
    run = FreqRunner(B, k_cap, int(cap.max()), **cfg)
    for _ in range(2):   # the second call finds the scratch as the first one left it
        min_prob = float(rng.choice([0.0, 0.1, 0.34, 0.5, 1.0]))
        max_occ = int(rng.choice([1, 2, 5, 100, 128]))
        got = run(flat, off, cap, ln, K, min_prob, max_occ)
        want = O.lookup_freq(flat, off, cap, ln, K, k_cap=k_cap, min_prob=min_prob, max_occ=max_occ, nthreads=8, **cfg)
        check(got, want)
    run.close()


def planted(rng, n, n_occ, pat_len, vocab=10**6, branch=3, cont=12):
    """Large-vocabulary filler with one pattern planted n_occ times, each followed by a continuation
    drawn from `branch` alternatives that share prefixes of random length; the history ends with the
    pattern, so the occurrences are exactly the planted ones."""
    h = rng.integers(1000, vocab, n).astype(np.int32)
    pat = rng.integers(0, 500, pat_len).astype(np.int32)
    alts = rng.integers(500, 520, (branch, cont)).astype(np.int32)
    alts[:, : int(rng.integers(0, cont // 2))] = alts[0, : 1][0]
    slot = pat_len + cont + 2
    places = rng.choice((n - 2 * slot) // slot, n_occ, replace=False) * slot + 1
    for p in places:
        h[p:p + pat_len] = pat
        h[p + pat_len:p + pat_len + cont] = alts[int(rng.integers(0, branch))]
    h[n - pat_len:] = pat
    return h


@pytest.mark.parametrize("n,n_occ,max_occ", [(3000, 7, 128), (20000, 128, 128), (20000, 129, 128), (20000, 60, 59),
                                             (70000, 100, 100), (9000, 128, 127)])
def test_planted_branches_across_chunks(n, n_occ, max_occ):
    rng = np.random.default_rng(n + n_occ)
    hs = [planted(rng, n - 17 * i, n_occ, int(rng.integers(2, 9))) for i in range(5)]
    flat, off, cap, ln = pack(hs, extra_cap=1)
    K = np.array([12, 64, 3, 40, 9], np.int32)
    run = FreqRunner(8, 64, int(cap.max()), spec_factor=4.0)
    for min_prob in (0.1, 0.4):
        got = run(flat, off, cap, ln, K, min_prob, max_occ)
        want = O.lookup_freq(flat, off, cap, ln, K, k_cap=64, spec_factor=4.0, min_prob=min_prob, max_occ=max_occ,
                             nthreads=8)
        check(got, want)
        assert (want.match_cnt == n_occ).all()
        assert want.draft_len.max() >= 3
        if n_occ <= max_occ and min_prob == 0.1:
            assert (want.score < want.draft_len).any()      # real branching: some probability below one
    run.close()


def test_workload_histories_and_selection():
    """Template-copy histories; a short maximum match length gives several occurrences per request,
    whose continuations differ where a copy was mutated."""
    w = W.CONFIGS["C2"].scaled(B=24, n=12000)
    rq = W.make_requests(w)
    cfg = dict(l_max=2, spec_factor=8.0)
    run = FreqRunner(rq.B, w.k_cap, int(rq.hist_cap.max()), **cfg)
    args = (rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K)
    for max_occ, thr, md, ml in ((128, 15.8, rq.model_draft, rq.model_len), (3, 15.8, rq.model_draft, rq.model_len),
                                 (128, 15.8, None, None)):
        got = run(*args, 0.1, max_occ, threshold=thr, model_draft=md, model_len=ml)
        want = O.lookup_freq(*args, k_cap=w.k_cap, min_prob=0.1, max_occ=max_occ, nthreads=8, **cfg)
        check(got, want)
        sel, sd, sl = O.freq_select(want, thr, md, ml)
        G.assert_equal("select", got["select"], sel)
        G.assert_equal("sel_draft", got["sel_draft"], sd)
        G.assert_equal("sel_len", got["sel_len"], sl)
        assert 0 < sel.sum() < rq.B
        assert want.match_cnt.max() >= 5 and (want.score < want.draft_len).any()
    # the configured match length (64): long matches, mostly a single occurrence each
    run.close()
    run = FreqRunner(rq.B, w.k_cap, int(rq.hist_cap.max()))
    check(run(*args, 0.1, 128), O.lookup_freq(*args, k_cap=w.k_cap, min_prob=0.1, max_occ=128, nthreads=8))
    run.close()


def test_degenerate_histories_and_bad_arguments():
    import paper_2606_01019_b200 as H
    hs = [[], [5], [5, 5], [5, 5, 5], [1, 2, 1, 2, 1, 2, 1], [9] * 500, list(range(50)), [3, 4, 3, 4]]
    flat, off, cap, ln = pack(hs)
    K = np.full(len(hs), 4, np.int32)
    run = FreqRunner(len(hs), 4, 500, min_match=1)
    for max_occ in (1, 128):
        got = run(flat, off, cap, ln, K, 0.1, max_occ)
        want = O.lookup_freq(flat, off, cap, ln, K, k_cap=4, min_match=1, min_prob=0.1, max_occ=max_occ)
        check(got, want)
    bad_ln = ln.copy(); bad_ln[4] = -3; bad_ln[6] = 10**6   # unusable lengths read as empty histories
    got = run(flat, off, cap, bad_ln, K, 0.1, 128, n_max=500)
    want = O.lookup_freq(flat, off, cap, bad_ln, K, k_cap=4, min_match=1, min_prob=0.1, max_occ=128)
    check(got, want)
    assert got["draft_len"][4] == 0 and got["draft_len"][6] == 0 and got["score"][6] == 0.0
    with pytest.raises(H.HvdError):
        run(flat, off, cap, ln, K, 0.1, 129)
    with pytest.raises(H.HvdError):
        run(flat, off, cap, ln, K, 0.1, 0)
    run.close()
