"""hvd_verify_commit_prefix on the GPU: verification that reads the logits only up to the window that holds the
first rejected draft token.  Every output, the histories and the state must equal the oracle's full
verification (array by array, target_tok aside) and the oracle's own row-by-row prefix walk, and the number of
rows streamed must be the walk's."""
import dataclasses
import os

import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from oracle import pipeline as P
from tests import gpu_helpers as G
from tests.test_gpu_edge_cases import hand_requests, small

pytestmark = pytest.mark.gpu


def boundary_bytes():
    """What the library under test was told (the variable is read when a context is created)."""
    return int(os.environ.get("HVD_PREFIX_BOUNDARY_BYTES", O.PREFIX_BOUNDARY_BYTES))


@pytest.fixture(autouse=True, params=["every window", "windows by size"])
def window_rule(request, monkeypatch):
    """Every case twice: with a boundary worth of one byte, so that small inputs are cut into all their windows
    ([0,2), [2,4), [4,8), ...), and with the library's own rule (small inputs: one window)."""
    if request.param == "every window":
        monkeypatch.setenv("HVD_PREFIX_BOUNDARY_BYTES", "1")
    else:
        monkeypatch.delenv("HVD_PREFIX_BOUNDARY_BYTES", raising=False)


def oracle_prefix(w, rq, sc, logits_np):
    dtype = O.F32 if w.dtype == "f32" else O.BF16
    return O.verify_commit_prefix(logits_np, dtype, w.V, rq.row_off, 0, sc.sel_draft, sc.sel_len, sc.select,
                                  k_cap=w.k_cap, hist=rq.hist, hist_off=rq.hist_off, hist_cap=rq.hist_cap,
                                  hist_len=rq.hist_len, state=rq.state, boundary_bytes=boundary_bytes())


def compare(g, vf, rq_after):
    for k in ("accepted", "committed", "n_commit", "status"):
        G.assert_equal(k, g[k], getattr(vf, k))
    G.assert_equal("hist_len", g["hist_len"], rq_after.hist_len)
    G.assert_equal("hist (all slabs and guard words)", g["hist"], rq_after.hist)
    G.assert_equal("state.sel_bits", g["state"]["sel_bits"], rq_after.state["sel_bits"])
    G.assert_equal("state.acc_ring", g["state"]["acc_ring"], rq_after.state["acc_ring"])
    assert (g["hist"][rq_after.guard_mask] == W.GUARD_VALUE).all()


def run_prefix(inp, rq=None, steps=1, ctx=None, salt0=700):
    """`steps` decoding steps with the prefix verification on the GPU, the oracle's chain beside it (full
    verification on one copy of the requests, prefix walk on another); returns the rows streamed per step."""
    import torch
    w = inp.w
    rq_full = inp.rq.copy() if rq is None else rq.copy()
    rq_walk = rq_full.copy()
    own = ctx is None
    ctx = ctx or G.make_ctx(w, rq_full)
    G.set_predictor(ctx, inp)
    batch = G.make_batch(ctx, w, rq_full)
    rows = torch.zeros(1, dtype=torch.int64, device="cuda")
    seen = []
    for s in range(steps):
        if s == 0:
            lg, lg_np = inp.logits, inp.logits_np
        else:                                      # fresh logits that agree with this step's selection for a while
            lk = P.lookup(w, rq_full, 8)
            sc = P.score_select(w, rq_full, lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, 8, inp.Wh, inp.bh)
            lg = W.make_logits(w, int(rq_full.row_off[-1]), device="cuda", salt=salt0 + s)
            W.plant_agreement(w, lg, rq_full.row_off, sc.sel_draft, sc.sel_len, W.make_agreement(w, sc.sel_len), salt=salt0 + s)
            lg_np = W.logits_to_numpy(lg)
        if lg.device.type != "cuda":
            lg = lg.cuda()
        batch.lookup_score_select()
        before = int(rows.item())
        batch.verify_commit_prefix(lg, rows)
        g = batch.download()
        assert ctx.hvd_device_status() == 0
        out = P.step(inp, rq_full, nthreads=P.host_threads(), logits_np=lg_np)       # the definition, all rows
        G.compare_lookup(g, out.lk)
        assert G.compare_score(g, out.sc, inp.tau).all()
        compare(g, out.vf, rq_full)
        walk = oracle_prefix(w, rq_walk, out.sc, lg_np)                              # the row-by-row walk
        compare(g, walk, rq_walk)
        assert int(rows.item()) - before == walk.rows_read, (int(rows.item()) - before, walk.rows_read)
        seen.append((walk.rows_read, walk.rows_needed, int((out.sc.sel_len.astype(np.int64) + 1).sum())))
    if own:
        ctx.close()
    return seen


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", dict(B=24, n=9000, V=20011)), ("C4", dict(B=6, n=40000, V=5003)),
                                     ("C5", dict(B=61, n=(40, 9000), V=32003)), ("C3", dict(B=40, n=4096, V=40009))])
def test_scaled_workloads(name, kw):
    w = W.CONFIGS[name].scaled(**kw) if kw else W.CONFIGS[name]
    seen = run_prefix(P.prepare(w, device="cuda"), steps=3)
    for read, needed, full in seen:
        assert needed <= read <= full


@pytest.mark.parametrize("name", ["C2", "C3", "C5"])
def test_full_size(name):
    w = W.CONFIGS[name]
    (read, needed, full), = run_prefix(P.prepare(w, device="cuda"))
    print(f"{name}: rows needed by the results {needed}, streamed {read}, read by the full verification {full}")
    assert read < 0.6 * full


@pytest.mark.parametrize("k_cap", [1, 2, 3, 4, 8, 33, 64])
def test_every_accepted_length(k_cap):
    """One request per (draft length, accepted length) pair, ragged rows: every window edge is crossed."""
    import torch
    w = small(V=211, k_cap=k_cap)
    rng = np.random.default_rng(k_cap)
    pairs = [(m, a) for m in range(k_cap + 1) for a in sorted({0, 1, 2, 3, 4, 7, 8, 15, 16, 31, 32, m - 1, m}) if 0 <= a <= m]
    B = len(pairs)
    hists = [rng.integers(0, 5, 300 + 3 * i) for i in range(B)]
    drafts = rng.integers(0, w.V, (B, k_cap)).astype(np.int32)
    rq = hand_requests(w, hists, [m for m, _ in pairs], model_len=[m for m, _ in pairs], model_draft=drafts,
                       cap_extra=[int(rng.choice([0, 1, 3, k_cap + 1, 4 * (k_cap + 1)])) for _ in pairs])
    wb = w.scaled(B=B)
    inp = P.prepare(wb, device="cuda", rq=rq)
    # selection as the oracle makes it, then logits that accept exactly pairs[b][1] tokens where the draft allows
    lk = P.lookup(wb, rq.copy(), 8)
    sc = P.score_select(wb, rq.copy(), lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, 8)
    A = np.minimum(np.array([a for _, a in pairs], np.int32), sc.sel_len)
    lg = W.make_logits(wb, int(rq.row_off[-1]), device="cuda", salt=9)
    W.plant_agreement(wb, lg, rq.row_off, sc.sel_draft, sc.sel_len, A, salt=9)
    inp = dataclasses.replace(inp, logits=lg, logits_np=W.logits_to_numpy(lg))
    run_prefix(inp, rq=rq)


def test_bad_lengths_capacity_and_odd_draft_tokens():
    w = small()
    rng = np.random.default_rng(7)
    hists = [rng.integers(0, 3, 500) for _ in range(12)]
    extra = [9, 5, 4, 3, 2, 1, 0, 9, 9, 9, 9, 0]
    hist_len = [500, 500, 500, 500, 500, 500, 500, -1, 510, 2**31 - 1, 500, 500]
    md = rng.integers(0, w.V, (12, w.k_cap)).astype(np.int32)
    md[10, 0] = -1; md[11, 1] = w.V            # draft tokens outside the vocabulary never match
    rq = hand_requests(w, hists, [8] * 12, cap_extra=extra, hist_len=hist_len, model_draft=md)
    inp = P.prepare(w.scaled(B=rq.B), device="cuda", rq=rq)
    run_prefix(inp, rq=rq)


def test_prefix_and_full_calls_share_one_context():
    """The two entry points in turn on one context and one batch: scratch (row keys, unit counters, alive flags)
    must be back at rest after each."""
    import torch
    w = W.CONFIGS["C2"].scaled(B=16, n=4096, V=50021)
    inp = P.prepare(w, device="cuda")
    rq = inp.rq.copy()
    ctx = G.make_ctx(w, rq)
    G.set_predictor(ctx, inp)
    batch = G.make_batch(ctx, w, rq)
    for s in range(6):
        lk = P.lookup(w, rq, 8)
        sc = P.score_select(w, rq, lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, 8)
        lg = W.make_logits(w, int(rq.row_off[-1]), device="cuda", salt=80 + s)
        W.plant_agreement(w, lg, rq.row_off, sc.sel_draft, sc.sel_len, W.make_agreement(w, sc.sel_len), salt=80 + s)
        batch.lookup_score_select()
        if s % 2 == 0:
            batch.verify_commit_prefix(lg)
        else:
            batch.verify_commit(lg)
        g = batch.download()
        vf = P.verify_commit(w, rq, sc, W.logits_to_numpy(lg), 8)
        compare(g, vf, rq)
        if s % 2:
            G.assert_equal("target_tok", g["target_tok"], vf.target_tok)
    assert ctx.hvd_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("B,n", [(24, 3000), (10, 30000), (6, 50000)])
def test_chain_without_host_synchronisation(B, n):
    """Six steps enqueued back to back on one stream, each verified by the prefix form (no host synchronisation
    in between: the lookup of a step may be resident while the windows of the step before are still streaming):
    final histories, lengths, states and the last step's outputs must equal the oracle's chain."""
    import torch
    w = W.CONFIGS["C2"].scaled(B=B, n=n, V=5003)
    inp = P.prepare(w, device="cuda")
    S = 6
    rq_o = inp.rq.copy()
    logits_dev, outs = [], []
    for s in range(S):
        lk = P.lookup(w, rq_o, 8)
        sc = P.score_select(w, rq_o, lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, 8, inp.Wh, inp.bh)
        lg = W.make_logits(w, int(rq_o.row_off[-1]), device="cuda", salt=300 + s)
        W.plant_agreement(w, lg, rq_o.row_off, sc.sel_draft, sc.sel_len, W.make_agreement(w, sc.sel_len), salt=300 + s)
        vf = P.verify_commit(w, rq_o, sc, W.logits_to_numpy(lg), 8)
        logits_dev.append(lg)
        outs.append((lk, sc, vf))
    rq_g = inp.rq.copy()
    ctx = G.make_ctx(w, rq_g)
    G.set_predictor(ctx, inp)
    batch = G.make_batch(ctx, w, rq_g)
    rows = torch.zeros(1, dtype=torch.int64, device="cuda")
    torch.cuda.synchronize()
    for s in range(S):
        batch.lookup_score_select()
        batch.verify_commit_prefix(logits_dev[s], rows)
    g = batch.download()
    lk, sc, vf = outs[-1]
    G.compare_lookup(g, lk)
    assert G.compare_score(g, sc, inp.tau).all()
    compare(g, vf, rq_o)
    assert ctx.hvd_device_status() == 0 and int(rows.item()) > 0
    ctx.close()


def test_random_batches():
    from tests.test_gpu_random_sweep import draw_case
    for it in range(60):
        rng = np.random.default_rng(3100000 + it)
        w, rq = draw_case(rng, it)
        inp = P.prepare(w, device="cuda", rq=rq)
        try:
            run_prefix(inp, rq=rq, steps=2)
        except AssertionError as e:
            raise AssertionError(f"case {it} (B {w.B}, k_cap {w.k_cap}, V {w.V}, {w.dtype}): {e}")


def test_host_side_argument_errors():
    import torch
    import paper_2606_01019_b200 as H
    w = W.CONFIGS["C1"]
    inp = P.prepare(w, device="cuda")
    ctx = G.make_ctx(w, inp.rq)
    b = G.make_batch(ctx, w, inp.rq)
    odd = torch.zeros(3, dtype=torch.int32, device="cuda")[1:]        # 4-byte aligned only
    with pytest.raises(H.HvdError, match="rows_read"):
        ctx.hvd_verify_commit_prefix(b.B, inp.logits, b.dtype, b.V, b.row_off, b.k_uniform, b.total_rows, b.sel_draft,
                                     b.sel_len, b.select, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.state,
                                     b.accepted, b.committed, b.n_commit, odd, b.status)
    with pytest.raises(H.HvdError, match="NULL"):
        ctx.hvd_verify_commit_prefix(b.B, None, b.dtype, b.V, b.row_off, b.k_uniform, b.total_rows, b.sel_draft,
                                     b.sel_len, b.select, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.state,
                                     b.accepted, b.committed, b.n_commit, None, b.status)
    ctx.close()
