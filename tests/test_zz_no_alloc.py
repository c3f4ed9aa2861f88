"""hvd_verify_commit_noalloc: the verification entry point for callers that cannot allocate
(its scratch memory is a static array inside the library).  Called through the C ABI and checked
against hvd_verify_commit on the same inputs and, in the first round, against the CPU oracle's
verification of the same selection, for two calls in a row, so that whatever the first call leaves
in the shared array must not disturb the second.  Collected last on purpose."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import pipeline as P
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu

OUTPUTS = ("accepted", "committed", "n_commit", "target_tok", "status", "hist", "hist_len")


def run_both(w, rounds=2):
    import torch
    import paper_2606_01019_b200 as H
    inp = P.prepare(w, device="cuda")
    ctx = G.make_ctx(w, inp.rq)
    ctx.hvd_set_predictor(inp.W1, inp.b1, inp.W2, inp.b2, inp.tau)
    ref = G.make_batch(ctx, w, inp.rq.copy())      # existing entry point, context scratch
    new = G.make_batch(ctx, w, inp.rq.copy())      # new entry point, static scratch
    dtype = H.F32 if w.dtype == "f32" else H.BF16
    for r in range(rounds):
        logits = inp.logits if r == 0 else W.make_logits(w, int(inp.rq.row_off[-1]), device="cuda", salt=7 + r)
        for b in (ref, new):                       # both sides get their draft from the same kernels
            b.lookup()
            b.score_select()
        ref.verify_commit(logits)
        H.hvd_verify_commit_noalloc(new.B, ctx.k_cap, logits, dtype, w.V, new.row_off, new.k_uniform,
                                    new.total_rows, new.sel_draft, new.sel_len, new.select, new.hist,
                                    new.hist_off, new.hist_cap, new.hist_len, new.state, new.accepted,
                                    new.committed, new.n_commit, new.target_tok, new.status)
        torch.cuda.synchronize()
        a, b = ref.download(), new.download()
        if r == 0:
            # the oracle on the other side as well: its verification of the selection the kernels made
            # (the selection itself is compared with the oracle's in the parity tests)
            rq_o = inp.rq.copy()
            sel = type("Sel", (), dict(sel_draft=b["sel_draft"], sel_len=b["sel_len"], select=b["select"]))
            vf = P.verify_commit(w, rq_o, sel, inp.logits_np, nthreads=P.host_threads())
            G.compare_verify(b, vf, rq_o)
        for k in OUTPUTS:                          # integer results: bit-exact, as in the other tests
            G.assert_equal(f"round {r}: {k}", b[k], a[k])
        G.assert_equal(f"round {r}: acc_ring", b["state"]["acc_ring"], a["state"]["acc_ring"])
        G.assert_equal(f"round {r}: sel_bits", b["state"]["sel_bits"], a["state"]["sel_bits"])
        assert (b["n_commit"] >= 1).all()
    ctx.close()


def test_noalloc_matches_context_entry_point_fp32():
    run_both(W.CONFIGS["C1"])


def test_noalloc_matches_context_entry_point_bf16_ragged():
    run_both(W.CONFIGS["C5"].scaled(B=40, n=(64, 3000), V=32003))


def test_noalloc_beyond_160_mb_of_logits():
    """More than 160 MB of logits.  Row blocks of equal height (816 rows of 128 256 bf16: 209 MB): the kernel whose
    grid is (batch, row of the block, request).  Ragged row blocks (48 requests with 5 to 33 rows, about 230 MB):
    the persistent kernel, whose unit counters and their reset then run on the static array too."""
    run_both(W.CONFIGS["C2"].scaled(B=48, n=1024))
    w = W.CONFIGS["C5"].scaled(B=48, n=(64, 3000))
    assert int(W.make_requests(w).row_off[-1]) * w.V * w.elt > 160 * 2**20
    run_both(w)


def test_noalloc_rejects_sizes_beyond_the_static_array():
    import torch
    import paper_2606_01019_b200 as H
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    s = torch.zeros(8, dtype=torch.int64, device="cuda")
    lg = torch.zeros(16, dtype=torch.float32, device="cuda")
    rows = H.NOALLOC_MAX_ROWS + 1
    with pytest.raises(H.HvdError, match="HVD_NOALLOC_MAX_ROWS"):
        H.hvd_verify_commit_noalloc(1, 4, lg, H.F32, 4, s, 0, rows, z, z, z, z, s, z, z, s, z, z, z, None, z)
    with pytest.raises(H.HvdError, match="HVD_NOALLOC_MAX_BATCH"):
        H.hvd_verify_commit_noalloc(H.NOALLOC_MAX_BATCH + 1, 4, lg, H.F32, 4, s, 0, 4, z, z, z, z, s, z, z, s, z, z,
                                    z, None, z)
