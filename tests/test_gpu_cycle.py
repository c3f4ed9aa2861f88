"""GPU parity of hvd_verify_commit_next: the commit of one cycle and the lookup, features, score and
selection of the next one in one call, against the oracle's chain of separate steps."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import pipeline as P
from tests import gpu_helpers as G
from tests.test_gpu_edge_cases import hand_requests, small

pytestmark = pytest.mark.gpu


def oracle_chain(inp, rq, S, salt=500):
    """S cycles of the oracle on rq (updated in place), the logits of every cycle planted to agree with that
    cycle's selected draft, and the lookup + selection that follows the last commit."""
    w = inp.w
    nt = P.host_threads()
    logits, outs = [], []
    for s in range(S):
        lk = P.lookup(w, rq, nt)
        sc = P.score_select(w, rq, lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, nt, inp.Wh, inp.bh)
        A = W.make_agreement(w, sc.sel_len)
        lg = W.make_logits(w, int(rq.row_off[-1]), device="cuda", salt=salt + s)
        W.plant_agreement(w, lg, rq.row_off, sc.sel_draft, sc.sel_len, A, salt=salt + s)
        vf = P.verify_commit(w, rq, sc, W.logits_to_numpy(lg), nt)
        logits.append(lg)
        outs.append((lk, sc, vf, rq.copy()))
    lk = P.lookup(w, rq, nt)
    sc = P.score_select(w, rq, lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, nt, inp.Wh, inp.bh)
    return logits, outs, (lk, sc)


def run_chain(inp, rq0, S, check_every_cycle=True, ctx_over=None):
    import torch
    w = inp.w
    logits, outs, last = oracle_chain(inp, rq0.copy(), S)
    rq_g = rq0.copy()
    ctx = G.make_ctx(w, rq_g, **(ctx_over or {}))
    G.set_predictor(ctx, inp)
    batch = G.make_batch(ctx, w, rq_g)
    batch.lookup_score_select()
    grew = np.zeros(rq0.B, bool)
    for s in range(S):
        batch.verify_commit_next(logits[s])
        if check_every_cycle or s == S - 1:
            g = batch.download()
            lk_n, sc_n = (outs[s + 1][0], outs[s + 1][1]) if s + 1 < S else last
            G.compare_verify(g, outs[s][2], outs[s][3])          # this cycle's commit
            G.compare_lookup(g, lk_n)                            # the next cycle's lookup ...
            same = G.compare_score(g, sc_n, inp.tau)             # ... and selection
            assert same.all()
            grew |= outs[s][2].n_commit > 0
    torch.cuda.synchronize()
    assert ctx.hvd_device_status() == 0
    ctx.close()
    return grew


@pytest.mark.parametrize("name,kw", [
    ("C1", {}),                                              # fp32 logits, 2 K tokens
    ("C2", dict(B=24, n=900, V=5003)),                       # the smallest CTA shape
    ("C2", dict(B=24, n=3000, V=5003)),
    ("C2", dict(B=20, n=7000, V=20011)),
    ("C2", dict(B=12, n=16384, V=20011)),                    # the benchmark's history length
    ("C2", dict(B=6, n=32700, V=5003)),                      # the longest histories one CTA takes
    ("C5", dict(B=60, n=(2, 5000), V=32003)),                # ragged lengths and draft caps
])
def test_chain_of_cycles(name, kw):
    inp = P.prepare(W.CONFIGS[name].scaled(**kw), device="cuda")
    grew = run_chain(inp, inp.rq, 5)
    assert grew.any()


def test_full_size_c2():
    """The benchmark's workload at full size (64 histories of 16 384 tokens, vocabulary 128 256)."""
    inp = P.prepare(W.CONFIGS["C2"], device="cuda")
    grew = run_chain(inp, inp.rq, 3)
    assert grew.all()


def test_chain_without_host_synchronisation():
    inp = P.prepare(W.CONFIGS["C2"].scaled(B=24, n=3000, V=5003), device="cuda")
    run_chain(inp, inp.rq, 6, check_every_cycle=False)


@pytest.mark.parametrize("kw", [dict(B=5, n=33000, V=5003), dict(B=4, n=70000, V=5003)])
def test_long_histories_take_the_separate_kernels(kw):
    inp = P.prepare(W.CONFIGS["C2"].scaled(**kw), device="cuda")
    run_chain(inp, inp.rq, 3)


def test_two_layer_predictor_takes_the_separate_kernels():
    inp = P.prepare(W.CONFIGS["C2"].scaled(B=16, n=4000, V=5003, hidden=64, hidden_layers=2), device="cuda")
    run_chain(inp, inp.rq, 3)


@pytest.mark.parametrize("mis", [1, 2, 3])
def test_misaligned_slabs(mis):
    w = small()
    rng = np.random.default_rng(40 + mis)
    base = rng.integers(0, 4, 5000)
    hists = [base[: 1000 + 211 * i] for i in range(10)] + [rng.integers(0, w.V, 2047 + i) for i in range(4)]
    rq = hand_requests(w, hists, [8] * len(hists), misalign=[mis] * len(hists))
    inp = P.prepare(w.scaled(B=rq.B), device="cuda", rq=rq)
    run_chain(inp, rq, 4)


def test_tiny_full_and_invalid_requests():
    """Histories of 0..5 tokens, slabs with no room or room for part of a commit (the history then grows by
    less than the commit, or not at all), and lengths outside the slab (request skipped by the commit and
    looked up as an empty history)."""
    w = small()
    rng = np.random.default_rng(44)
    hists = [rng.integers(0, 3, n) for n in (0, 1, 2, 3, 4, 5, 40, 41, 300, 301, 302, 303, 1500, 1501)]
    B = len(hists)
    extra = [36] * B
    extra[8], extra[9], extra[10], extra[11] = 0, 1, 2, 5
    lens = [len(h) for h in hists]
    lens[12] = -3
    lens[13] = len(hists[13]) + 100
    rq = hand_requests(w, hists, [8] * B, cap_extra=extra, hist_len=lens)
    inp = P.prepare(w.scaled(B=B), device="cuda", rq=rq)
    run_chain(inp, rq, 4)


def test_commit_next_equals_the_two_calls():
    """One cycle, the same inputs: hvd_verify_commit_next against hvd_verify_commit followed by
    hvd_lookup_score_select, array by array."""
    inp = P.prepare(W.CONFIGS["C2"].scaled(B=32, n=5000, V=20011), device="cuda")
    w = inp.w
    res = []
    for fused in (False, True):
        rq = inp.rq.copy()
        ctx = G.make_ctx(w, rq)
        G.set_predictor(ctx, inp)
        batch = G.make_batch(ctx, w, rq)
        batch.lookup_score_select()
        if fused:
            batch.verify_commit_next(inp.logits)
        else:
            batch.verify_commit(inp.logits)
            batch.lookup_score_select()
        res.append(batch.download())
        ctx.close()
    for k in res[0]:
        a, b = res[0][k], res[1][k]
        if k in ("freq_score", "match_src", "features_ext"):
            continue
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8)), k


def test_host_side_argument_errors():
    import paper_2606_01019_b200 as H
    w = small()
    rng = np.random.default_rng(46)
    rq = hand_requests(w, [rng.integers(0, 4, 200) for _ in range(3)], [8] * 3)
    inp = P.prepare(w.scaled(B=3), device="cuda", rq=rq)
    ctx = G.make_ctx(w, rq)
    b = G.make_batch(ctx, w, rq)
    with pytest.raises(H.HvdError, match="hvd_set_predictor first"):
        b.verify_commit_next(inp.logits)
    G.set_predictor(ctx, inp)
    b.lookup_score_select()
    with pytest.raises(H.HvdError, match="go together"):
        b.ctx.hvd_verify_commit_next(b.B, inp.logits, b.dtype, b.V, b.row_off, b.k_uniform, b.total_rows, b.sel_draft,
                                     b.sel_len, b.select, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.state,
                                     b.accepted, b.committed, b.n_commit, None, b.status, K=b.K, n_max=b.n_max,
                                     prompt_len=b.prompt_len, model_draft=b.model_draft, model_len=None,
                                     draft=b.draft, draft_len=b.draft_len, match_len=b.match_len,
                                     match_pos=b.match_pos, match_cnt=b.match_cnt, features=None, score=b.score,
                                     next_select=b.select, next_sel_draft=b.sel_draft, next_sel_len=b.sel_len)
    with pytest.raises(H.HvdError, match="NULL pointer in next"):
        b.ctx.hvd_verify_commit_next(b.B, inp.logits, b.dtype, b.V, b.row_off, b.k_uniform, b.total_rows, b.sel_draft,
                                     b.sel_len, b.select, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.state,
                                     b.accepted, b.committed, b.n_commit, None, b.status, K=b.K, n_max=b.n_max,
                                     prompt_len=b.prompt_len, model_draft=None, model_len=None,
                                     draft=b.draft, draft_len=b.draft_len, match_len=b.match_len,
                                     match_pos=b.match_pos, match_cnt=b.match_cnt, features=None, score=None,
                                     next_select=b.select, next_sel_draft=b.sel_draft, next_sel_len=b.sel_len)
    with pytest.raises(H.HvdError, match="n_max"):
        b.ctx.hvd_verify_commit_next(b.B, inp.logits, b.dtype, b.V, b.row_off, b.k_uniform, b.total_rows, b.sel_draft,
                                     b.sel_len, b.select, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.state,
                                     b.accepted, b.committed, b.n_commit, None, b.status, K=b.K, n_max=10**7,
                                     prompt_len=b.prompt_len, model_draft=None, model_len=None,
                                     draft=b.draft, draft_len=b.draft_len, match_len=b.match_len,
                                     match_pos=b.match_pos, match_cnt=b.match_cnt, features=None, score=b.score,
                                     next_select=b.select, next_sel_draft=b.sel_draft, next_sel_len=b.sel_len)
    import torch
    torch.cuda.synchronize()
    assert ctx.hvd_device_status() == 0
    ctx.close()
