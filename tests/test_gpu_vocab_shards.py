"""Verification with the vocabulary split into shards (a vocabulary-parallel output layer): per-shard
row keys from hvd_verify_keys, their element-wise maximum (what an all-reduce with MAX computes;
the shards run here as independent launches on one GPU), hvd_commit_keys -- against the oracle's
verification of the whole rows, bit for bit."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from oracle import pipeline as P
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu


def run_sharded(inp, bounds):
    import torch
    import paper_2606_01019_b200 as H
    from paper_2606_01019_b200.sharding import reduce_keys_over_ranks
    w, rq = inp.w, inp.rq.copy()
    ctx = G.make_ctx(w, rq)
    G.set_predictor(ctx, inp)
    batch = G.make_batch(ctx, w, rq)
    batch.lookup_score_select()
    logits = inp.logits.cuda() if inp.logits.device.type != "cuda" else inp.logits
    rows = batch.total_rows
    full = logits.reshape(-1)[: rows * w.V].reshape(rows, w.V)
    keys = None
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        shard = full[:, lo:hi].contiguous()                       # this "rank's" slice of every row
        k = torch.full((rows,), 12345, dtype=torch.int64, device="cuda")
        ctx.hvd_verify_keys(batch.B, shard, batch.dtype, int(hi - lo), int(lo), batch.row_off, batch.k_uniform, rows,
                            batch.sel_len, batch.hist_len, batch.hist_cap, k)
        keys = k if keys is None else torch.maximum(keys, k)      # the MAX all-reduce
    reduce_keys_over_ranks(keys)                                  # identity without a process group
    ctx.hvd_commit_keys(batch.B, keys, w.V, batch.row_off, batch.k_uniform, rows, batch.sel_draft, batch.sel_len,
                        batch.select, batch.hist, batch.hist_off, batch.hist_cap, batch.hist_len, batch.state,
                        batch.accepted, batch.committed, batch.n_commit, batch.target_tok, batch.status)
    g = batch.download()
    # the context's own scratch must be at rest: a plain verification on the same context still works
    ctx.close()
    return g


@pytest.mark.parametrize("name,kw,shards", [("C1", {}, 2), ("C1", {}, 3), ("C2", dict(B=9, n=3000, V=20011), 4),
                                            ("C2", dict(B=9, n=3000, V=20011), 1), ("C5", dict(B=40, n=(64, 3000), V=32003), 8),
                                            ("C2", dict(B=5, n=2000, V=9), 3)])
def test_sharded_vocabulary_equals_whole_rows(name, kw, shards):
    w = W.CONFIGS[name].scaled(**kw)
    inp = P.prepare(w, device="cuda")
    bounds = [int(x) for x in (np.arange(shards + 1) * w.V) // shards]
    g = run_sharded(inp, bounds)
    rq = inp.rq.copy()
    out = P.step(inp, rq, nthreads=8)
    G.compare_lookup(g, out.lk)
    same = G.compare_score(g, out.sc, inp.tau)
    assert same.all()
    G.compare_verify(g, out.vf, rq)


def test_ties_across_shards_and_uneven_shards():
    """Equal maxima in different shards (the lower global index wins), a maximum at a shard's first and
    last entry, -0.0 against +0.0 across shards, uneven shard sizes."""
    import torch
    w = W.CONFIGS["C1"].scaled(B=4, n=600, V=1000)
    inp = P.prepare(w, device="cuda")
    lg = inp.logits.reshape(-1)[: int(inp.rq.row_off[-1]) * w.V].reshape(-1, w.V)
    lg[0, :] = -1.0; lg[0, 333] = 40.0; lg[0, 334] = 40.0; lg[0, 900] = 40.0
    lg[1, :] = -2.0; lg[1, 999] = 40.0
    lg[2, :] = -0.0; lg[2, 700] = 0.0                             # all equal: index 0
    lg[3, :] = -5.0; lg[3, 334] = 41.0; lg[3, 0] = 41.0
    inp.logits_np = W.logits_to_numpy(inp.logits)
    for bounds in ([0, 334, 1000], [0, 1, 333, 334, 999, 1000], [0, 500, 1000]):
        g = run_sharded(inp, bounds)
        rq = inp.rq.copy()
        out = P.step(inp, rq, nthreads=4)
        G.compare_verify(g, out.vf, rq)
        r0 = int(inp.rq.row_off[0])
        assert list(g["target_tok"][r0:r0 + 1]) == [333] or inp.rq.row_off[0] != 0
