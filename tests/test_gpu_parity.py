"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer results bit-exact; fp32 scores within 1e-5 relative."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from oracle import pipeline as P
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu


def test_c1_full():
    inp = P.prepare(W.CONFIGS["C1"], device="cuda")
    g, out, _ = G.run_and_compare(inp)
    assert (g["accepted"] == inp.A)[inp.strict].all()
    assert g["select"].sum() > 0


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", dict(B=24, n=9000, V=20011)), ("C4", dict(B=6, n=40000, V=5003)),
                                     ("C5", dict(B=60, n=(2, 5000), V=32003))])
def test_fused_lookup_score_select(name, kw):
    """hvd_lookup_score_select gives what hvd_lookup followed by hvd_score_select gives."""
    inp = P.prepare(W.CONFIGS[name].scaled(**kw), device="cuda")
    G.run_and_compare(inp, fused=True)


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("name,kw", [("C2", dict(B=40, n=6000, V=20011, hidden=256, hidden_layers=2)),
                                     ("C1", dict(hidden=64, hidden_layers=2)),
                                     ("C5", dict(B=33, n=(8, 3000), V=32003, hidden=200, hidden_layers=2))])
def test_two_hidden_layer_predictor(name, kw, fused):
    """The paper's predictor shape (two hidden ReLU layers): scores within 1e-5, same selections."""
    inp = P.prepare(W.CONFIGS[name].scaled(**kw), device="cuda")
    g, out, _ = G.run_and_compare(inp, fused=fused)
    assert 0 < out.sc.select.sum() < len(out.sc.select)


def test_switching_between_one_and_two_layers_on_one_context():
    w2 = W.CONFIGS["C1"].scaled(hidden=32, hidden_layers=2)
    w1 = W.CONFIGS["C1"]
    inp2, inp1 = P.prepare(w2, device="cuda"), P.prepare(w1, device="cuda")
    ctx = G.make_ctx(w1, inp1.rq)
    for inp in (inp2, inp1, inp2):
        G.set_predictor(ctx, inp)
        batch = G.make_batch(ctx, inp.w, inp.rq.copy())
        G.run_and_compare(inp, ctx=ctx, batch=batch, rq=inp.rq.copy())
    ctx.close()


def test_c1_uniform_row_layout():
    inp = P.prepare(W.CONFIGS["C1"], device="cuda")
    G.run_and_compare(inp, uniform_rows=True)


@pytest.mark.parametrize("name", ["C2", "C3", "C4", "C5"])
def test_full_size_configs(name):
    """Every request, row and token of the full-size workloads, in the launch configuration the
    benchmark uses (same context limits, same entry points)."""
    inp = P.prepare(W.CONFIGS[name], device="cuda")
    g, out, _ = G.run_and_compare(inp, fused=True)      # the entry points the benchmark times
    assert (g["accepted"] == inp.A)[inp.strict].all()
    sel = g["select"]
    assert 0 < sel.sum() < len(sel)                       # both draft sources in play
    assert (g["status"] == O.REQ_OK).all()


@pytest.mark.parametrize("name,kw", [
    ("C2", dict(B=7, n=5000, V=20011)),                    # odd V: rows not 16-byte multiples (bf16)
    ("C2", dict(B=5, n=3000, V=9)),
    ("C1", dict(B=3, n=700, V=4099)),                      # fp32, odd V
    ("C1", dict(B=3, n=700, V=1)),
    ("C1", dict(B=2, n=300, V=7)),
    ("C2", dict(B=3, n=1500, V=8)),
    ("C3", dict(B=9, n=2500, V=151936)),
    ("C5", dict(B=40, n=(16, 3000), V=32003)),
])
def test_scaled_shapes(name, kw):
    inp = P.prepare(W.CONFIGS[name].scaled(**kw), device="cuda")
    G.run_and_compare(inp)


def test_multi_step_loop_and_scratch_reuse():
    """Eight chained steps on one context and one device batch: histories keep growing, the
    scratch memory must be back at rest after every call."""
    for name, kw in (("C1", {}), ("C2", dict(B=16, n=4096, V=50021))):
        w = W.CONFIGS[name].scaled(**kw)
        inp = P.prepare(w, device="cuda")
        rq = inp.rq.copy()
        batch = None
        ctx = G.make_ctx(w, rq)
        ctx.hvd_set_predictor(inp.W1, inp.b1, inp.W2, inp.b2, inp.tau)
        for s in range(8):
            logits = W.make_logits(w, int(rq.row_off[-1]), device="cuda", salt=50 + s)
            if batch is None:
                batch = G.make_batch(ctx, w, rq)
            g, out, batch = G.run_and_compare(inp, ctx=ctx, logits=logits, logits_np=W.logits_to_numpy(logits),
                                              rq=rq, batch=batch)
        assert (rq.hist_len > inp.rq.hist_len).all()
        ctx.close()


@pytest.mark.parametrize("pinned", [False, True])
@pytest.mark.parametrize("boundary", [None, "1"])
def test_host_buffer_entry_point(boundary, pinned, monkeypatch):
    """hvd_step_host: same step with host arrays in and out (copies inside the call).  The logits are copied and
    verified window by window; small inputs have one window, so every case runs once more with a window boundary
    worth one byte (rows [0,2), [2,4), [4,9) for the draft cap of 8).  The second call gets other logits: a row
    that this call leaves on the host must not be read from what an earlier call left in the staging area.
    Pageable logits are staged window by window; page-locked ones are read in place by the streaming kernels."""
    if boundary is not None:
        monkeypatch.setenv("HVD_PREFIX_BOUNDARY_BYTES", boundary)
    import paper_2606_01019_b200 as H
    from tests.test_gpu_edge_cases import hand_requests, small
    rng = np.random.default_rng(77)
    we = small()
    hists = [rng.integers(0, 3, n) for n in (0, 1, 5, 300, 301, 302, 1500, 1501, 2000)]
    lens = [len(h) for h in hists]
    lens[6], lens[7] = -2, len(hists[7]) + 500             # lengths outside the slab: no logits rows are copied
    rq_e = hand_requests(we, hists, [8] * len(hists), cap_extra=[36, 36, 36, 0, 1, 3, 36, 36, 36], hist_len=lens)
    cases = [(W.CONFIGS["C1"], None, False), (W.CONFIGS["C5"].scaled(B=24, n=(64, 3000), V=20011), None, False),
             (we.scaled(B=rq_e.B), rq_e, False), (we.scaled(B=rq_e.B), rq_e, True)]
    for w, rq_given, uniform in cases:
        inp = P.prepare(w, device="cpu", rq=rq_given)
        rq_g, rq_o = inp.rq.copy(), inp.rq.copy()
        ctx = G.make_ctx(w, rq_g)
        ctx.hvd_set_predictor(inp.W1, inp.b1, inp.W2, inp.b2, inp.tau)
        B, kc = rq_g.B, w.k_cap
        o = dict(score=np.zeros(B, np.float32), select=np.zeros(B, np.int32), sel_draft=np.zeros((B, kc), np.int32),
                 sel_len=np.zeros(B, np.int32), accepted=np.zeros(B, np.int32),
                 committed=np.zeros((B, kc + 1), np.int32), n_commit=np.zeros(B, np.int32),
                 status=np.zeros(B, np.int32))
        for rep in range(2):       # second call: staging area reused, histories have grown
            lg_np = inp.logits_np if rep == 0 else np.ascontiguousarray(np.roll(inp.logits_np.reshape(-1, w.V), 1, axis=1))
            lg_host = lg_np
            if pinned:
                import torch
                lg_host = torch.from_numpy(lg_np.view(np.int16) if lg_np.dtype == np.uint16 else lg_np).pin_memory()
            ctx.hvd_step_host(B=B, n_max=int(rq_g.hist_cap.max()), hist=rq_g.hist, hist_off=rq_g.hist_off,
                              hist_cap=rq_g.hist_cap, hist_len=rq_g.hist_len, K=rq_g.K, prompt_len=rq_g.prompt_len,
                              state=rq_g.state, model_draft=rq_g.model_draft, model_len=rq_g.model_len,
                              logits=lg_host, dtype=H.F32 if w.dtype == "f32" else H.BF16, V=w.V,
                              row_off=None if uniform else rq_g.row_off, k_uniform=w.k_cap if uniform else 0,
                              total_rows=int(rq_g.row_off[-1]), **o)
            out = P.step(inp, rq_o, logits_np=lg_np)
            G.assert_equal("score", o["score"], out.sc.score)
            for k in ("select", "sel_draft", "sel_len"):
                G.assert_equal(k, o[k], getattr(out.sc, k))
            for k in ("accepted", "committed", "n_commit", "status"):
                G.assert_equal(k, o[k], getattr(out.vf, k))
            G.assert_equal("hist", rq_g.hist, rq_o.hist)
            G.assert_equal("hist_len", rq_g.hist_len, rq_o.hist_len)
            G.assert_equal("acc_ring", rq_g.state["acc_ring"], rq_o.state["acc_ring"])
            G.assert_equal("sel_bits", rq_g.state["sel_bits"], rq_o.state["sel_bits"])
        ctx.close()


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("B,n", [(24, 3000), (24, 12000), (10, 30000), (6, 50000), (20, 70000)])
def test_chained_steps_without_host_synchronisation(fused, B, n):
    """Six steps enqueued back to back on one stream (no host synchronisation in between, so the kernels of
    consecutive steps overlap as far as programmatic dependent launch lets them): the final histories,
    lengths, states and the last step's outputs must equal the oracle's chain.  The longer histories take the
    lookup shapes that read the slab layout and ask the L2 for the slab while the previous step's commit may
    still be appending to it (one CTA of 1024 threads per request; clusters of 8 and 16 chunk CTAs)."""
    import torch
    w = W.CONFIGS["C2"].scaled(B=B, n=n, V=5003)
    inp = P.prepare(w, device="cuda")
    S = 6
    # the oracle's chain first: it fixes the logits of every step (each agrees with that step's selected draft)
    rq_o = inp.rq.copy()
    logits_dev, outs = [], []
    for s in range(S):
        lk = P.lookup(w, rq_o, 8)
        sc = P.score_select(w, rq_o, lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, 8, inp.Wh, inp.bh)
        A = W.make_agreement(w, sc.sel_len)
        lg = W.make_logits(w, int(rq_o.row_off[-1]), device="cuda", salt=300 + s)
        W.plant_agreement(w, lg, rq_o.row_off, sc.sel_draft, sc.sel_len, A, salt=300 + s)
        vf = P.verify_commit(w, rq_o, sc, W.logits_to_numpy(lg), 8)
        logits_dev.append(lg)
        outs.append((lk, sc, vf))
    # the same chain on the GPU, enqueued in one go
    rq_g = inp.rq.copy()
    ctx = G.make_ctx(w, rq_g)
    G.set_predictor(ctx, inp)
    batch = G.make_batch(ctx, w, rq_g)
    torch.cuda.synchronize()
    for s in range(S):
        batch.step(logits_dev[s], fused=fused)
    g = batch.download()
    lk, sc, vf = outs[-1]
    G.compare_lookup(g, lk)
    same = G.compare_score(g, sc, inp.tau)
    assert same.all()
    G.compare_verify(g, vf, rq_o)
    assert (rq_o.hist_len > inp.rq.hist_len).all()
    ctx.close()
