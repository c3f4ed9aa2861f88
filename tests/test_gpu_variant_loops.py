"""Chained decoding steps that combine the variants of the path on one context and one device batch,
against the same chain in the oracle: (A) the frequency-based hybrid rule, (B) shared warm-up
corpus + extended feature vector + two hidden layers.  Every output of every step is compared; the
histories, lengths and recent-history states must agree after each commit."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu
f32 = np.float32


def oracle_verify(w, rq, sel_draft, sel_len, select, logits_np):
    return O.verify_commit(logits_np, O.BF16 if w.dtype == "bf16" else O.F32, w.V, rq.row_off, 0, sel_draft, sel_len,
                           select, k_cap=w.k_cap, hist=rq.hist, hist_off=rq.hist_off, hist_cap=rq.hist_cap,
                           hist_len=rq.hist_len, state=rq.state, nthreads=8)


def fresh_logits(w, rq, sel_draft, sel_len, step):
    """Logits whose row maxima agree with the selected drafts for a seeded number of tokens."""
    A = W.make_agreement(w, sel_len)
    logits = W.make_logits(w, int(rq.row_off[-1]), device="cuda", salt=900 + step)
    W.plant_agreement(w, logits, rq.row_off, sel_draft, sel_len, A, salt=900 + step)
    return logits, W.logits_to_numpy(logits)


@pytest.mark.parametrize("name,kw,l_max", [("C2", dict(B=20, n=3000, V=30011), 2), ("C5", dict(B=48, n=(200, 4000), V=20011), 64)])
def test_frequency_hybrid_loop(name, kw, l_max):
    w = W.CONFIGS[name].scaled(**kw)
    rq = W.make_requests(w)
    cfg = dict(l_max=l_max, min_match=min(w.min_match, l_max), spec_factor=8.0)
    ctx = G.make_ctx(w, rq, **cfg)
    batch = G.make_batch(ctx, w, rq)
    accepted_total = 0
    for step in range(5):
        fq = O.lookup_freq(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, k_cap=w.k_cap, min_prob=0.1, max_occ=128,
                           nthreads=8, **cfg)
        thr = float(f32(np.median(fq.score[fq.draft_len > 0]))) if (fq.draft_len > 0).any() else 1.0
        sel, sd, sl = O.freq_select(fq, thr, rq.model_draft, rq.model_len)
        logits, logits_np = fresh_logits(w, rq, sd, sl, step)
        batch.lookup_freq(0.1, 128, thr)
        batch.verify_commit(logits)
        vf = oracle_verify(w, rq, sd, sl, sel, logits_np)
        g = batch.download()
        G.compare_lookup(g, fq)
        G.assert_equal("freq score bits", g["freq_score"].view(np.uint32), fq.score.view(np.uint32))
        for k, v in (("select", sel), ("sel_draft", sd), ("sel_len", sl)):
            G.assert_equal(k, g[k], v)
        G.compare_verify(g, vf, rq)
        accepted_total += int(vf.accepted.sum())
    assert accepted_total > 0
    ctx.close()


@pytest.mark.parametrize("name,kw", [("C5", dict(B=40, n=(100, 3000), V=20011, hidden=256)), ("C3", dict(B=12, n=2500, V=9001, hidden=32))])
def test_corpus_and_extended_features_loop(name, kw):
    import torch
    w = W.CONFIGS[name].scaled(**kw)
    rq = W.make_requests(w)
    corpus = W.make_corpus(w, n_traces=12, trace_len=(512, 4096))
    rng = np.random.default_rng(8)
    cls = rng.integers(0, 32, w.V).astype(np.uint8)
    H = w.hidden
    two = H == 256
    W1 = rng.normal(0, 0.1, (H, 14)).astype(f32); b1 = rng.normal(0, 0.1, H).astype(f32); W2 = rng.normal(0, 0.1, H).astype(f32)
    Wh = rng.normal(0, 0.1, (H, H)).astype(f32) if two else None
    bh = rng.normal(0, 0.1, H).astype(f32) if two else None
    ctx = G.make_ctx(w, rq)
    corpus_d, cls_d = torch.as_tensor(corpus, device="cuda"), torch.as_tensor(cls, device="cuda")
    ctx.hvd_set_corpus(corpus_d)
    ctx.hvd_set_token_classes(cls_d)
    batch = G.make_batch(ctx, w, rq)
    from_corpus = 0
    for step in range(4):
        lk = O.lookup_corpus(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, corpus, k_cap=w.k_cap, l_max=w.l_max,
                             min_match=w.min_match, nthreads=8)
        kw_sc = dict(k_cap=w.k_cap, W1=W1, b1=b1, W2=W2, b2=w.b2, Wh=Wh, bh=bh, nthreads=8, match_src=lk.match_src)
        pre = O.score_select_ext(rq.hist_len, rq.prompt_len, rq.state, rq.K, lk, None, cls, rq.model_draft, rq.model_len,
                                 tau=0.0, **kw_sc)
        has = lk.draft_len > 0
        tau = float(f32(np.median(pre.score64[has]))) if has.any() else 0.0
        sc = O.score_select_ext(rq.hist_len, rq.prompt_len, rq.state, rq.K, lk, None, cls, rq.model_draft, rq.model_len,
                                tau=tau, **kw_sc)
        ctx.hvd_set_predictor_ext(W1, b1, W2, w.b2, tau, Wh, bh)      # a new threshold every step
        logits, logits_np = fresh_logits(w, rq, sc.sel_draft, sc.sel_len, step)
        batch.lookup_corpus()
        batch.score_select_ext(src=True)
        batch.verify_commit(logits)
        g = batch.download()
        G.compare_lookup(g, lk)
        G.assert_equal("match_src", g["match_src"], lk.match_src)
        g["features"] = g["features_ext"]
        same = G.compare_score(g, sc, tau)
        assert same.all(), "selection differs inside the tau band: the rest of the step is not comparable"
        vf = oracle_verify(w, rq, sc.sel_draft, sc.sel_len, sc.select, logits_np)
        G.compare_verify(g, vf, rq)
        from_corpus += int(lk.match_src.sum())
    assert from_corpus > 0 or name != "C5"
    ctx.close()


@pytest.mark.parametrize("name", ["C2", "C3", "C4", "C5"])
def test_variants_at_full_size(name):
    """The frequency-weighted lookup and the corpus lookup on the full-size request batches."""
    import torch
    w = W.CONFIGS[name]
    rq = W.make_requests(w)
    ctx = G.make_ctx(w, rq)
    batch = G.make_batch(ctx, w, rq)
    args = (rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K)
    batch.lookup_freq(0.1, 128, 2.0)
    g = batch.download()
    fq = O.lookup_freq(*args, k_cap=w.k_cap, l_max=w.l_max, min_match=w.min_match, min_prob=0.1, max_occ=128, nthreads=16)
    G.compare_lookup(g, fq)
    G.assert_equal("freq score bits", g["freq_score"].view(np.uint32), fq.score.view(np.uint32))
    sel, sd, sl = O.freq_select(fq, 2.0, rq.model_draft, rq.model_len)
    for k, v in (("select", sel), ("sel_draft", sd), ("sel_len", sl)):
        G.assert_equal(k, g[k], v)
    corpus = W.make_corpus(w, n_traces=64)
    corpus_d = torch.as_tensor(corpus, device="cuda")
    ctx.hvd_set_corpus(corpus_d)
    batch.lookup_corpus()
    g = batch.download()
    lk = O.lookup_corpus(*args, corpus, k_cap=w.k_cap, l_max=w.l_max, min_match=w.min_match, nthreads=16)
    G.compare_lookup(g, lk)
    G.assert_equal("match_src", g["match_src"], lk.match_src)
    ctx.close()


def test_variants_at_the_maximum_batch():
    """8192 requests (the largest batch a context takes) with short histories through every variant entry
    point: grids, per-request scratch and the 16-requests-per-cluster scoring at their limits."""
    import torch
    from tests.test_gpu_edge_cases import hand_requests, small
    B = 8192
    w = small(V=61, k_cap=8, hidden=256).scaled(B=B)
    rng = np.random.default_rng(21)
    hists = [rng.integers(0, 4, int(n)) for n in rng.integers(0, 90, B)]
    rq = hand_requests(w, hists, rng.integers(0, 9, B))
    ctx = G.make_ctx(w, rq)
    batch = G.make_batch(ctx, w, rq)
    args = (rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K)
    kw = dict(k_cap=w.k_cap, l_max=w.l_max, min_match=w.min_match, nthreads=16)
    # frequency-weighted lookup with selection
    batch.lookup_freq(0.1, 128, 3.0)
    g = batch.download()
    fq = O.lookup_freq(*args, min_prob=0.1, max_occ=128, **kw)
    G.compare_lookup(g, fq)
    G.assert_equal("freq score bits", g["freq_score"].view(np.uint32), fq.score.view(np.uint32))
    sel, sd, sl = O.freq_select(fq, 3.0, rq.model_draft, rq.model_len)
    for k, v in (("select", sel), ("sel_draft", sd), ("sel_len", sl)):
        G.assert_equal(k, g[k], v)
    # corpus lookup
    corpus = np.concatenate([rng.integers(0, 4, 3000), [-1], rng.integers(0, 4, 2000)]).astype(np.int32)
    corpus_d = torch.as_tensor(corpus, device="cuda")
    ctx.hvd_set_corpus(corpus_d)
    batch.lookup_corpus()
    g = batch.download()
    lk = O.lookup_corpus(*args, corpus, **kw)
    G.compare_lookup(g, lk)
    G.assert_equal("match_src", g["match_src"], lk.match_src)
    # extended features, two hidden layers (sixteen requests per cluster)
    cls = rng.integers(0, 32, w.V).astype(np.uint8)
    H = w.hidden
    W1 = rng.normal(0, 0.1, (H, 14)).astype(f32); b1 = rng.normal(0, 0.1, H).astype(f32); W2 = rng.normal(0, 0.1, H).astype(f32)
    Wh = rng.normal(0, 0.1, (H, H)).astype(f32); bh = rng.normal(0, 0.1, H).astype(f32)
    cls_d = torch.as_tensor(cls, device="cuda")
    ctx.hvd_set_token_classes(cls_d)
    ctx.hvd_set_predictor_ext(W1, b1, W2, 6.0, 6.0, Wh, bh)
    batch.score_select_ext(src=True)
    g = batch.download()
    sc = O.score_select_ext(rq.hist_len, rq.prompt_len, rq.state, rq.K, lk, None, cls, rq.model_draft, rq.model_len,
                            k_cap=w.k_cap, W1=W1, b1=b1, W2=W2, b2=6.0, tau=6.0, Wh=Wh, bh=bh, nthreads=16, match_src=lk.match_src)
    g["features"] = g["features_ext"]
    G.compare_score(g, sc, 6.0)
    ctx.close()
