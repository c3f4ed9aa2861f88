"""GPU parity of the trace-replay labeller against the oracle."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu


def gpu_replay(x, K, k_cap, max_batch=1024, **cfg):
    import torch
    import paper_2606_01019_b200 as H
    n = len(x)
    ctx = H.Context(max_batch=max_batch, k_cap=k_cap, max_hist_len=max(n, 1), max_rows=1, max_vocab=1, **cfg)
    xd = torch.as_tensor(np.ascontiguousarray(x, np.int32), device="cuda")
    outs = [torch.full((n,), -12345, dtype=torch.int32, device="cuda") for _ in range(5)]
    ctx.hvd_replay_labels(xd, n, K, *outs)
    torch.cuda.synchronize()
    res = [o.cpu().numpy() for o in outs]
    ctx.close()
    return res


@pytest.mark.parametrize("n,vocab,K,k_cap,max_batch", [(1, 3, 4, 4, 8), (2, 1, 4, 4, 8), (57, 2, 3, 8, 16), (700, 3, 8, 8, 256),
                                                       (3000, 4, 16, 16, 1024), (5000, 50000, 64, 64, 4096)])
def test_replay_random_traces(n, vocab, K, k_cap, max_batch):
    x = np.random.default_rng(n).integers(0, vocab, n)
    got = gpu_replay(x, K, k_cap, max_batch)
    want = O.replay_labels(x, K, k_cap=k_cap, nthreads=8)
    for name, g, w in zip(("label", "draft_len", "match_len", "match_pos", "match_cnt"), got,
                          (want.label, want.draft_len, want.match_len, want.match_pos, want.match_cnt)):
        G.assert_equal(name, g, w)


def test_replay_workload_history_and_repeated_document():
    rq = W.make_requests(W.CONFIGS["C2"].scaled(B=2, n=6000))
    D = np.random.default_rng(5).permutation(10**6)[:900].astype(np.int32)
    for x in (rq.history(1), np.concatenate([D, D, D[:300]])):
        got = gpu_replay(x, 16, 16, 2048)
        want = O.replay_labels(x, 16, k_cap=16, nthreads=8)
        for name, g, w in zip(("label", "draft_len", "match_len", "match_pos", "match_cnt"), got,
                              (want.label, want.draft_len, want.match_len, want.match_pos, want.match_cnt)):
            G.assert_equal(name, g, w)
        assert got[0].max() >= 8


@pytest.mark.parametrize("n", [255, 256, 257, 258, 511, 513, 1025, 4097])
@pytest.mark.parametrize("cfg", [dict(min_match=1, l_max=64), dict(min_match=3, l_max=5), dict(min_match=2, l_max=2, spec_factor=2.5),
                                 dict(min_match=2, l_max=64, spec_factor=0.5, spec_offset=1.0)])
def test_replay_segment_boundaries_and_rules(n, cfg):
    """Trace lengths around the 256-state segments and 256-diagonal blocks of the kernel, with the match
    and draft-length rules varied; small vocabularies make runs cross the boundaries."""
    rng = np.random.default_rng(n)
    x = np.concatenate([rng.integers(0, 2, n // 2), rng.integers(0, 50, n - n // 2)])
    got = gpu_replay(x, 7, 8, 64, **cfg)
    want = O.replay_labels(x, 7, k_cap=8, nthreads=8, **cfg)
    for name, g, w in zip(("label", "draft_len", "match_len", "match_pos", "match_cnt"), got,
                          (want.label, want.draft_len, want.match_len, want.match_pos, want.match_cnt)):
        G.assert_equal(name, g, w)


def test_replay_two_traces_on_one_context():
    """The scratch grows with the longer trace and is back at rest after every call."""
    import torch
    import paper_2606_01019_b200 as H
    rng = np.random.default_rng(3)
    ctx = H.Context(max_batch=8, k_cap=8, max_hist_len=6000, max_rows=1, max_vocab=1)
    for n in (300, 6000, 1200, 6000):
        x = rng.integers(0, 3, n).astype(np.int32)
        xd = torch.as_tensor(x, device="cuda")
        outs = [torch.full((n,), -12345, dtype=torch.int32, device="cuda") for _ in range(5)]
        ctx.hvd_replay_labels(xd, n, 8, *outs)
        torch.cuda.synchronize()
        want = O.replay_labels(x, 8, k_cap=8, nthreads=8)
        for name, g, w in zip(("label", "draft_len", "match_len", "match_pos", "match_cnt"), outs,
                              (want.label, want.draft_len, want.match_len, want.match_pos, want.match_cnt)):
            G.assert_equal(name, g.cpu().numpy(), w)
    ctx.close()
