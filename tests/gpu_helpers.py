"""Shared pieces of the GPU parity tests: run the CUDA path through the binding and compare every
output and in/out array with the oracle's, element by element."""
import numpy as np

import hvd_workloads as W
from oracle import pipeline as P

SCORE_RTOL = 1e-5      # fp32 payoff scores: relative tolerance stated by the benchmark spec
TAU_BAND = 1e-4        # selections may differ only inside this band around tau


def make_ctx(w, rq, **over):
    import paper_2606_01019_b200 as H
    kw = dict(max_batch=rq.B, k_cap=w.k_cap, max_hist_len=max(int(rq.hist_cap.max()), 1),
              max_rows=max(int(rq.row_off[-1]), 1), max_vocab=w.V, l_max=w.l_max, min_match=w.min_match,
              hidden=w.hidden)
    kw.update(over)
    return H.Context(**kw)


def set_predictor(ctx, inp):
    if inp.Wh is not None:
        ctx.hvd_set_predictor2(inp.W1, inp.b1, inp.Wh, inp.bh, inp.W2, inp.b2, inp.tau)
    else:
        ctx.hvd_set_predictor(inp.W1, inp.b1, inp.W2, inp.b2, inp.tau)


def make_batch(ctx, w, rq, uniform_rows=False):
    from paper_2606_01019_b200.runner import DeviceBatch
    return DeviceBatch(ctx, hist=rq.hist, hist_off=rq.hist_off, hist_cap=rq.hist_cap, hist_len=rq.hist_len,
                       K=rq.K, prompt_len=rq.prompt_len, state=rq.state, model_draft=rq.model_draft,
                       model_len=rq.model_len, row_off=rq.row_off, V=w.V, dtype=w.dtype,
                       uniform_rows=uniform_rows)


def assert_equal(name, got, want):
    got, want = np.asarray(got), np.asarray(want)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    if not (got == want).all():
        bad = np.argwhere(got != want)
        i = tuple(bad[0])
        raise AssertionError(f"{name}: {len(bad)} mismatches, first at {i}: got {got[i]} want {want[i]}")


def compare_lookup(g, lk):
    for k in ("draft", "draft_len", "match_len", "match_pos", "match_cnt"):
        assert_equal(k, g[k], getattr(lk, k))


def compare_score(g, sc, tau):
    assert_equal("features", g["features"].view(np.uint32), sc.features.view(np.uint32))   # bit-exact
    rel = np.abs(g["score"].astype(np.float64) - sc.score.astype(np.float64)) / np.maximum(np.abs(sc.score64), 1e-30)
    assert rel.max() <= SCORE_RTOL, rel.max()
    outside = np.abs(sc.score64 - tau) > TAU_BAND
    assert_equal("select(outside band)", g["select"][outside], sc.select[outside])
    same = g["select"] == sc.select
    assert_equal("sel_len", g["sel_len"][same], sc.sel_len[same])
    assert_equal("sel_draft", g["sel_draft"][same], sc.sel_draft[same])
    return same


def compare_verify(g, vf, rq_after):
    for k in ("accepted", "committed", "n_commit", "target_tok", "status"):
        assert_equal(k, g[k], getattr(vf, k))
    assert_equal("hist_len", g["hist_len"], rq_after.hist_len)
    assert_equal("hist (all slabs and guard words)", g["hist"], rq_after.hist)
    assert_equal("state.sel_bits", g["state"]["sel_bits"], rq_after.state["sel_bits"])
    assert_equal("state.acc_ring", g["state"]["acc_ring"], rq_after.state["acc_ring"])
    assert (g["hist"][rq_after.guard_mask] == W.GUARD_VALUE).all()


def run_and_compare(inp, ctx=None, uniform_rows=False, logits=None, logits_np=None, rq=None, batch=None,
                    nthreads=None, fused=False):
    """One full step on the GPU and in the oracle from the same inputs; returns (gpu dict, StepOut)."""
    w = inp.w
    rq = inp.rq.copy() if rq is None else rq
    own = ctx is None
    if batch is None:
        if own:
            ctx = make_ctx(w, rq)
        set_predictor(ctx, inp)
        batch = make_batch(ctx, w, rq, uniform_rows)
    lg = inp.logits if logits is None else logits
    if lg.device.type != "cuda":
        lg = lg.cuda()
    batch.step(lg, fused=fused)
    g = batch.download()
    out = P.step(inp, rq, nthreads=nthreads or P.host_threads(), logits_np=logits_np)
    compare_lookup(g, out.lk)
    same = compare_score(g, out.sc, inp.tau)
    assert same.all(), "selection differs inside the tau band: the rest of the step is not comparable"
    compare_verify(g, out.vf, rq)
    if own:
        ctx.close()
    return g, out, batch
