"""Request sharding on the GPU path: the ragged workload cut into contiguous ranges of near-equal bytes
(sharding.partition_requests, what a rank of a data-parallel deployment would take), every range run through
the library as a batch of its own, and the concatenated results compared with the whole-batch run, which is
itself compared with the oracle.  One GPU: the ranges run one after the other, there is no collective."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import pipeline as P
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu

PER_REQUEST = ("draft", "draft_len", "match_len", "match_pos", "match_cnt", "select", "sel_draft", "sel_len",
               "accepted", "committed", "n_commit", "status", "hist_len")


@pytest.mark.parametrize("name,kw", [("C5", {}), ("C5", dict(B=61, n=(40, 9000), V=32003))])
def test_ranges_of_a_ragged_batch_equal_the_whole_batch(name, kw):
    from paper_2606_01019_b200.sharding import partition_requests, request_cost
    w = W.CONFIGS[name].scaled(**kw) if kw else W.CONFIGS[name]
    inp = P.prepare(w, device="cuda")
    whole, out, _ = G.run_and_compare(inp, fused=True)        # whole batch: GPU == oracle, array by array
    rq = inp.rq
    cost = request_cost(rq.hist_len, rq.K, w.V, w.elt)
    logits = inp.logits if inp.logits.device.type == "cuda" else inp.logits.cuda()
    for world in (2, 4, 8):
        bounds = partition_requests(cost, world)
        assert bounds[0] == 0 and bounds[-1] == rq.B and (np.diff(bounds) >= 0).all()
        share = np.array([cost[bounds[r]:bounds[r + 1]].sum() for r in range(world)], np.float64)
        balance = share.max() / share.mean()
        print(f"{w.name} x{world}: requests per range {np.diff(bounds).tolist()}, bytes max/mean {balance:.3f}")
        assert balance < 1.0 + 2.0 * cost.max() / share.mean()   # off by at most about one request either way
        hist_after = rq.hist.copy()                                # every range appends to its own slabs
        got = {k: [] for k in PER_REQUEST}
        state, score, target = [], [], []
        for r in range(world):
            lo, hi = int(bounds[r]), int(bounds[r + 1])
            if lo == hi:
                continue
            sub = W.subset_requests(rq, lo, hi)
            ctx = G.make_ctx(w, sub)
            G.set_predictor(ctx, inp)
            batch = G.make_batch(ctx, w, sub)
            r0, r1 = int(rq.row_off[lo]), int(rq.row_off[hi])
            batch.step(logits[r0:r1], fused=True)
            g = batch.download()
            ctx.close()
            for k in PER_REQUEST:
                got[k].append(g[k])
            state.append(g["state"]); score.append(g["score"]); target.append(g["target_tok"])
            for b in range(lo, hi):                                # the range's slabs, as it left them
                o, c = int(rq.hist_off[b]), int(rq.hist_cap[b])
                hist_after[o:o + c] = g["hist"][o:o + c]
        for k in PER_REQUEST:
            G.assert_equal(f"x{world} {k}", np.concatenate(got[k]), whole[k])
        G.assert_equal(f"x{world} score", np.concatenate(score).view(np.uint32), whole["score"].view(np.uint32))
        G.assert_equal(f"x{world} target_tok", np.concatenate(target), whole["target_tok"])
        st = np.concatenate(state)
        G.assert_equal(f"x{world} sel_bits", st["sel_bits"], whole["state"]["sel_bits"])
        G.assert_equal(f"x{world} acc_ring", st["acc_ring"], whole["state"]["acc_ring"])
        G.assert_equal(f"x{world} hist (all slabs and guard words)", hist_after, whole["hist"])
