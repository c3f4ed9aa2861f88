"""GPU parity of token-tree verification (hvd_verify_commit_tree) against the oracle."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu


def run_tree_case(w, salt=0):
    import torch
    import paper_2606_01019_b200 as H
    rq = W.make_requests(w)
    tok, par, cnt = W.make_tree_drafts(w, rq.K)
    A = W.make_agreement(w, np.minimum(cnt, 8))
    logits = W.make_logits(w, int(rq.row_off[-1]), device="cuda", salt=salt)
    depth = W.plant_tree_agreement(w, logits, rq.row_off, tok, par, cnt, A, salt=salt)
    select = np.zeros(rq.B, np.int32)
    # oracle
    ro = rq.copy()
    dtype = O.F32 if w.dtype == "f32" else O.BF16
    want = O.verify_commit(W.logits_to_numpy(logits), dtype, w.V, ro.row_off, 0, tok, cnt, select, k_cap=w.k_cap,
                           hist=ro.hist, hist_off=ro.hist_off, hist_cap=ro.hist_cap, hist_len=ro.hist_len,
                           state=ro.state, nthreads=8, parent=par)
    # GPU
    ctx = G.make_ctx(w, rq)
    b = G.make_batch(ctx, w, rq.copy())
    up = lambda a: torch.as_tensor(np.ascontiguousarray(a, np.int32), device="cuda")
    b.sel_draft, b.sel_len, b.select = up(tok), up(cnt), up(select)
    parent = up(par)
    ctx.hvd_verify_commit_tree(b.B, logits, b.dtype, w.V, b.row_off, 0, b.total_rows, b.sel_draft, b.sel_len, parent,
                               b.select, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.state, b.accepted,
                               b.committed, b.n_commit, b.target_tok, b.status)
    g = b.download()
    G.compare_verify(g, want, ro)
    assert (want.accepted == depth).all()          # the planted path is what gets accepted
    ctx.close()
    return want


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", dict(B=24, n=3000, V=20011, K=32, k_cap=32)),
                                     ("C4", dict(B=5, n=2000, V=5003)), ("C5", dict(B=50, n=(8, 2000), V=32003))])
def test_tree_verification(name, kw):
    want = run_tree_case(W.CONFIGS[name].scaled(**kw))
    assert want.accepted.max() >= 2


def test_chain_as_tree_equals_linear_entry_point():
    """parent[i] = i-1: hvd_verify_commit_tree must give what hvd_verify_commit gives."""
    import torch
    from oracle import pipeline as P
    w = W.CONFIGS["C2"].scaled(B=12, n=2000, V=9001)
    inp = P.prepare(w, device="cuda")
    ctx = G.make_ctx(w, inp.rq)
    ctx.hvd_set_predictor(inp.W1, inp.b1, inp.W2, inp.b2, inp.tau)
    a, b = G.make_batch(ctx, w, inp.rq.copy()), G.make_batch(ctx, w, inp.rq.copy())
    for x in (a, b):
        x.lookup(); x.score_select()
    a.verify_commit(inp.logits)
    chain = torch.arange(-1, w.k_cap - 1, dtype=torch.int32, device="cuda").repeat(b.B, 1).contiguous()
    ctx.hvd_verify_commit_tree(b.B, inp.logits, b.dtype, w.V, b.row_off, 0, b.total_rows, b.sel_draft, b.sel_len, chain,
                               b.select, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.state, b.accepted,
                               b.committed, b.n_commit, b.target_tok, b.status)
    ga, gb = a.download(), b.download()
    for k in ("accepted", "committed", "n_commit", "target_tok", "status", "hist", "hist_len"):
        G.assert_equal(k, gb[k], ga[k])
    ctx.close()
