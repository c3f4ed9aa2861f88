"""GPU parity of scoring on the extended feature vector (draft-structure token-class shares, suffix
score) against the oracle: features bit for bit, scores within the stated tolerance, selections
identical outside the band around tau."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu
f32 = np.float32


def ext_weights(w, seed, two_layers):
    rng = np.random.default_rng(seed)
    H = w.hidden
    W1 = rng.normal(0, 0.1, (H, 14)).astype(f32); b1 = rng.normal(0, 0.1, H).astype(f32)
    W2 = rng.normal(0, 0.1, H).astype(f32)
    Wh = rng.normal(0, 0.1, (H, H)).astype(f32) if two_layers else None
    bh = rng.normal(0, 0.1, H).astype(f32) if two_layers else None
    return W1, b1, W2, Wh, bh


def run_gpu(ctx, rq, lk, suffix, k_cap, with_model=True):
    import torch
    B = rq.B
    dev = lambda a: None if a is None else torch.as_tensor(np.ascontiguousarray(a), device="cuda")
    out = dict(features=torch.full((B, 14), -7.0, device="cuda"), score=torch.full((B,), -7.0, device="cuda"),
               select=torch.full((B,), -5, dtype=torch.int32, device="cuda"),
               sel_draft=torch.full((B, k_cap), -5, dtype=torch.int32, device="cuda"),
               sel_len=torch.full((B,), -5, dtype=torch.int32, device="cuda"))
    state = torch.as_tensor(np.ascontiguousarray(rq.state).view(np.uint8).reshape(B, 16), device="cuda")
    ctx.hvd_score_select_ext(B, dev(rq.hist_len), dev(rq.prompt_len), state, dev(rq.K), dev(lk.draft), dev(lk.draft_len),
                             dev(lk.match_len), dev(lk.match_pos), dev(lk.match_cnt), dev(suffix),
                             dev(rq.model_draft) if with_model else None, dev(rq.model_len) if with_model else None,
                             out["features"], out["score"], out["select"], out["sel_draft"], out["sel_len"])
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


@pytest.mark.parametrize("name,kw,two_layers", [("C2", dict(B=70, n=4000, V=6000), False),
                                                ("C2", dict(B=70, n=4000, V=6000, hidden=256), True),
                                                ("C4", dict(B=33, n=9000, V=3000), False),
                                                ("C4", dict(B=33, n=9000, V=3000, hidden=200), True),
                                                ("C5", dict(B=130, n=(64, 3000), hidden=7), False)])
def test_extended_scoring(name, kw, two_layers):
    import torch
    w = W.CONFIGS[name].scaled(**kw)
    rq = W.make_requests(w)
    rng = np.random.default_rng(w.B)
    fq = O.lookup_freq(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, k_cap=w.k_cap, l_max=3, spec_factor=30.0,
                       max_occ=128, nthreads=8)                       # short matches: several occurrences, real scores
    cls = rng.integers(0, 32, w.V).astype(np.uint8)
    cls[rng.random(w.V) < 0.5] = 0
    W1, b1, W2, Wh, bh = ext_weights(w, 5, two_layers)
    pre = O.score_select_ext(rq.hist_len, rq.prompt_len, rq.state, rq.K, fq, fq.score, cls, None, None, k_cap=w.k_cap,
                             W1=W1, b1=b1, W2=W2, b2=w.b2, tau=0.0, Wh=Wh, bh=bh, nthreads=8)
    tau = float(f32(np.median(pre.score64[fq.draft_len > 0])))      # about half the requests take the cache draft
    ctx = G.make_ctx(w, rq)
    cls_d = torch.as_tensor(cls, device="cuda")
    ctx.hvd_set_token_classes(cls_d)
    ctx.hvd_set_predictor_ext(W1, b1, W2, w.b2, tau, Wh, bh)
    for suffix, with_model in ((fq.score, True), (None, False)):
        got = run_gpu(ctx, rq, fq, suffix, w.k_cap, with_model)
        want = O.score_select_ext(rq.hist_len, rq.prompt_len, rq.state, rq.K, fq, suffix, cls,
                                  rq.model_draft if with_model else None, rq.model_len if with_model else None,
                                  k_cap=w.k_cap, W1=W1, b1=b1, W2=W2, b2=w.b2, tau=tau, Wh=Wh, bh=bh, nthreads=8)
        same = G.compare_score(got, want, tau)
        assert same.mean() > 0.9
        if suffix is not None:
            assert 0 < want.select.sum() < rq.B
        assert (want.features[:, 8:13] > 0).any() and (fq.draft_len > 32).any() == (w.k_cap > 32)
    ctx.close()


def test_predictor_kinds_do_not_mix():
    import torch
    import paper_2606_01019_b200 as H
    w = W.CONFIGS["C2"].scaled(B=8, n=2000, V=500)
    rq = W.make_requests(w)
    lk = O.lookup(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, k_cap=w.k_cap)
    W1, b1, W2, _, _ = ext_weights(w, 1, False)
    ctx = G.make_ctx(w, rq)
    ctx.hvd_set_predictor_ext(W1, b1, W2, 0.0, 1.0)
    with pytest.raises(H.HvdError):                      # no token classes registered
        run_gpu(ctx, rq, lk, None, w.k_cap)
    cls_d = torch.zeros(w.V, dtype=torch.uint8, device="cuda")
    ctx.hvd_set_token_classes(cls_d)
    run_gpu(ctx, rq, lk, None, w.k_cap)
    batch = G.make_batch(ctx, w, rq)
    with pytest.raises(H.HvdError):                      # the base entry points have no predictor of their own now
        batch.lookup_score_select()
    with pytest.raises(H.HvdError):
        batch.lookup(); batch.score_select()
    b1W1, bb1, bW2, bb2, btau = W.make_predictor(w)
    ctx.hvd_set_predictor(b1W1, bb1, bW2, bb2, btau)
    with pytest.raises(H.HvdError):                      # and the other way round
        run_gpu(ctx, rq, lk, None, w.k_cap)
    ctx.close()
