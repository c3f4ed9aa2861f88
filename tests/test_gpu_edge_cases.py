"""GPU parity on the degenerate and adversarial shapes of the path."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import hvd_oracle as O
from oracle import pipeline as P
from tests import gpu_helpers as G

pytestmark = pytest.mark.gpu


def hand_requests(w, hists, K, cap_extra=None, hist_len=None, model_len=None, misalign=None, seed=0,
                  model_draft=None):
    rng = np.random.default_rng(seed)
    B = len(hists)
    K = np.asarray(K, np.int64)
    n = np.asarray([len(h) for h in hists], np.int64)
    extra = 4 * (K + 1) if cap_extra is None else np.asarray(cap_extra, np.int64)
    cap = n + extra
    prompt_len = np.floor(n * rng.uniform(0.0, 1.0, B)).astype(np.int32)
    state = np.zeros(B, W.STATE_DTYPE)
    state["sel_bits"] = rng.integers(0, 2**32, B, dtype=np.uint64).astype(np.uint32)
    state["acc_ring"] = rng.integers(0, 2**63, B, dtype=np.uint64)
    if model_draft is None:
        model_draft = rng.integers(0, w.V, (B, w.k_cap)).astype(np.int32)
    if model_len is None:
        model_len = K
    return W.pack_requests([np.asarray(h, np.int32) for h in hists], K, cap, prompt_len, state, model_draft,
                           model_len, hist_len=hist_len, misalign=misalign)


def small(V=997, k_cap=8, dtype="bf16", **kw):
    return W.CONFIGS["C2"].scaled(V=V, k_cap=k_cap, K=k_cap, dtype=dtype, calibrate_cache_frac=0.5, **kw)


def run(w, rq, **kw):
    inp = P.prepare(w.scaled(B=rq.B), device="cuda", rq=rq)
    return G.run_and_compare(inp, **kw), inp


@pytest.mark.parametrize("fused", [False, True])
def test_tiny_histories(fused):
    w = small()
    rng = np.random.default_rng(3)
    hists = []
    for n in (0, 1, 2, 3, 4, 5, 63, 64, 65, 66, 127, 128, 129, 1023, 1024, 1025, 1026, 1027, 2050):
        hists.append(rng.integers(0, 3, n))                 # tiny vocabulary: matches everywhere
        hists.append(rng.integers(0, w.V, n))               # large vocabulary: rarely any match
    rq = hand_requests(w, hists, [8] * len(hists))
    (g, out, _), _ = run(w, rq, fused=fused)
    assert (out.lk.match_len > 0).sum() > 10


def test_draft_caps_k0_k1_k64():
    w = small(k_cap=64)
    rng = np.random.default_rng(4)
    base = rng.integers(0, 5, 3000)
    hists = [base[: 2000 + 17 * i] for i in range(12)]
    K = [0, 1, 64, 0, 1, 64, 2, 63, 33, 32, 31, 64]
    rq = hand_requests(w, hists, K)
    run(w, rq)


def test_all_equal_and_periodic_histories():
    w = small()
    hists = [[7] * 300, [7] * 64, [7] * 65, [7] * 66, [1, 2] * 200, [1, 2, 3] * 150, [1, 2] * 31 + [1],
             [5] * 2, [5] * 3, [4, 4, 9] * 400 + [4]]
    rq = hand_requests(w, hists, [8] * len(hists))
    (g, out, _), _ = run(w, rq)
    assert tuple(int(x[0]) for x in (out.lk.match_len, out.lk.match_pos, out.lk.match_cnt, out.lk.draft_len)) == (64, 299, 236, 1)


def test_match_touching_slab_start_and_end():
    w = small(V=50021)
    rng = np.random.default_rng(5)
    hs = []
    for L in (2, 5, 64, 70):
        h = rng.permutation(40000)[:1500].astype(np.int64) + 5
        h[-L:] = h[:L]                       # only match ends at e = L: touches index 0
        hs.append(h)
        h = rng.permutation(40000)[:1500].astype(np.int64) + 5
        h[-3:] = h[-3]                       # x x x: longest match (2) ends at e = n-1, a one-token draft
        hs.append(h)
    rq = hand_requests(w, hs, [8] * len(hs))
    (g, out, _), _ = run(w, rq)
    assert out.lk.match_pos[0] == 2 and out.lk.match_len[4] == 64
    assert out.lk.match_pos[1] == 1499 and out.lk.draft_len[1] == 1


@pytest.mark.parametrize("mis", [1, 2, 3])
def test_misaligned_slabs(mis):
    w = small()
    rng = np.random.default_rng(6)
    hists = [rng.integers(0, 4, n) for n in (10, 100, 1024, 1025, 3000, 4099)]
    rq = hand_requests(w, hists, [8] * len(hists), misalign=[mis, (mis + 1) % 4, mis, 0, mis, mis])
    run(w, rq)


def test_capacity_edges_and_bad_lengths():
    w = small()
    rng = np.random.default_rng(7)
    hists = [rng.integers(0, 3, 500) for _ in range(12)]
    extra = [9, 5, 4, 3, 2, 1, 0, 9, 9, 9, 9, 0]
    hist_len = [500, 500, 500, 500, 500, 500, 500, -1, 510, 2**31 - 1, 500, 500]
    rq = hand_requests(w, hists, [8] * 12, cap_extra=extra, hist_len=hist_len)
    run(w, rq.copy(), fused=True)
    (g, out, _), _ = run(w, rq)
    assert (out.vf.status == O.REQ_BAD_LEN).sum() == 3
    assert (out.vf.status == O.REQ_CAPACITY).sum() >= 1


@pytest.mark.parametrize("small_bytes", [None, "0"])
def test_row_offsets_outside_the_logits(small_bytes, monkeypatch):
    """A row_off entry below 0 or beyond total_rows: the request is skipped with HVD_REQ_BAD_LEN, nothing is read
    or written outside the logits, the row keys or target_tok, and the other requests are verified as usual
    (with the warp-per-batch kernel and with the persistent one)."""
    if small_bytes is not None:
        monkeypatch.setenv("HVD_VERIFY_SMALL_BYTES", small_bytes)
    w = small()
    rng = np.random.default_rng(21)
    hists = [rng.integers(0, 3, 400 + 10 * i) for i in range(9)]
    rq = hand_requests(w, hists, [8, 3, 8, 0, 5, 8, 8, 2, 8])
    inp = P.prepare(w.scaled(B=rq.B), device="cuda", rq=rq)
    good = rq.copy()
    (g0, out, _) = G.run_and_compare(inp, rq=good)            # the reference results, with valid offsets
    ctx = G.make_ctx(w, rq)
    G.set_predictor(ctx, inp)
    batch = G.make_batch(ctx, w, rq.copy())
    import torch
    bad = rq.row_off.copy()
    bad[0] = -3                      # request 0 starts before the array
    bad[-1] = rq.row_off[-1] + 5     # the last request ends beyond it
    batch.row_off = torch.as_tensor(bad, device="cuda")
    batch.step(inp.logits if inp.logits.device.type == "cuda" else inp.logits.cuda())
    g = batch.download()
    assert ctx.hvd_device_status() == 0
    ctx.close()
    B = rq.B
    skipped = np.zeros(B, bool); skipped[[0, B - 1]] = True
    assert (g["status"][skipped] == O.REQ_BAD_LEN).all()
    assert (g["accepted"][skipped] == 0).all() and (g["n_commit"][skipped] == 0).all()
    assert (g["committed"][skipped] == -1).all()
    assert (g["hist_len"][skipped] == rq.hist_len[skipped]).all()
    for k in ("accepted", "committed", "n_commit", "status", "hist_len"):
        G.assert_equal(k, g[k][~skipped], (g0[k])[~skipped])
    rows_ok = np.zeros(int(rq.row_off[-1]), bool)
    rows_ok[rq.row_off[1]:rq.row_off[B - 1]] = True
    G.assert_equal("target_tok", g["target_tok"][rows_ok], g0["target_tok"][rows_ok])
    assert (g["target_tok"][~rows_ok] == -12345).all()        # rows of the skipped requests: never written
    # histories: the skipped requests' slabs as before the call, the others as the reference run left them
    want = good.hist.copy()
    for b in (0, B - 1):
        o, c = int(rq.hist_off[b]), int(rq.hist_cap[b])
        want[o:o + c] = rq.hist[o:o + c]
    G.assert_equal("hist (all slabs and guard words)", g["hist"], want)


def test_model_draft_clamp_and_out_of_vocab_tokens():
    w = small(k_cap=16)
    rng = np.random.default_rng(8)
    hists = [rng.integers(0, w.V, 800) for _ in range(10)]          # hardly any cache draft: model path
    K = [4, 8, 16, 0, 3, 16, 16, 1, 2, 5]
    md = rng.integers(0, w.V, (10, 16)).astype(np.int32)
    md[5, 3] = -1; md[6, 0] = w.V; md[2, 15] = 2**31 - 1
    rq = hand_requests(w, hists, K, model_len=[9, 8, 16, 5, 0, 16, 16, 1, 40, -3], model_draft=md)
    run(w.scaled(calibrate_cache_frac=None), rq.copy(), fused=True)
    (g, out, _), _ = run(w.scaled(calibrate_cache_frac=None), rq)
    assert (out.sc.select == 0).all()


def test_no_model_drafter():
    """model_draft = NULL: requests whose cache draft is not selected verify an empty draft."""
    w = W.CONFIGS["C1"]
    inp = P.prepare(w, device="cuda")
    rq = inp.rq.copy()
    rq.model_len[:] = 0
    inp2 = P.prepare(w, device="cuda", rq=rq)
    ctx = G.make_ctx(w, rq)
    ctx.hvd_set_predictor(inp2.W1, inp2.b1, inp2.W2, inp2.b2, inp2.tau)
    batch = G.make_batch(ctx, w, inp2.rq.copy())
    batch.model_draft = None
    batch.model_len = None
    G.run_and_compare(inp2, ctx=ctx, batch=batch, rq=inp2.rq.copy())
    ctx.close()


@pytest.mark.parametrize("V,dtype", [(1, "bf16"), (7, "bf16"), (8, "bf16"), (9, "bf16"), (15, "bf16"), (17, "bf16"),
                                     (1, "f32"), (3, "f32"), (4, "f32"), (5, "f32"), (32000, "f32"),
                                     (8193 * 8, "bf16"), (16384 * 8 + 3, "bf16"), (151936, "bf16")])
def test_vocab_sizes(V, dtype):
    w = small(V=V, dtype=dtype, k_cap=4)
    rng = np.random.default_rng(V)
    hists = [rng.integers(0, min(V, 3), 200 + 13 * i) for i in range(6)]
    rq = hand_requests(w, hists, [4, 3, 2, 1, 0, 4])
    run(w, rq)


def test_constructed_argmax_ties_on_device():
    """Whole rows of equal values, +-0, +inf duplicates, maxima in the first and last slot, and a
    duplicate maximum straddling two work items."""
    import torch
    w = small(V=40000, k_cap=8)
    rng = np.random.default_rng(9)
    hists = [rng.integers(0, w.V, 300) for _ in range(9)]
    rq = hand_requests(w, hists, [8] * 9)
    inp = P.prepare(w.scaled(B=9, calibrate_cache_frac=None), device="cuda", rq=rq)
    lg = inp.logits
    r = rq.row_off
    lg[r[0]:r[1]] = 1.5                                   # all equal -> token 0
    lg[r[1]:r[2]] = -0.0; lg[r[1], 17] = 0.0              # -0 == +0 -> token 0
    lg[r[2]:r[3]] = -5.0; lg[r[2], 39999] = 3.0           # maximum in the last slot
    lg[r[3]:r[4]] = -5.0; lg[r[3], 0] = 3.0               # maximum in the first slot
    lg[r[4], 16383] = float("inf"); lg[r[4], 16384] = float("inf")     # equal maxima across items
    lg[r[5], 30000] = 40.0; lg[r[5], 20] = 40.0           # equal maxima far apart
    lg[r[6]:r[7]] = float("-inf")                         # nothing but -inf -> token 0
    lg[r[7]:r[8]] = -0.0                                  # nothing but -0
    inp.logits_np = W.logits_to_numpy(lg)
    g, out, _ = G.run_and_compare(inp)
    t = out.vf.target_tok
    assert t[r[0]] == 0 and t[r[1]] == 0 and t[r[2]] == 39999 and t[r[3]] == 0
    assert t[r[4]] == 16383 and t[r[5]] == 20 and t[r[6]] == 0 and t[r[7]] == 0


def test_batch_of_one_and_full_context_batch():
    w = small()
    rng = np.random.default_rng(10)
    rq = hand_requests(w, [rng.integers(0, 3, 777)], [8])
    run(w, rq)
    hists = [rng.integers(0, 4, int(n)) for n in rng.integers(0, 600, 700)]
    rq = hand_requests(w, hists, rng.integers(0, 9, 700))
    run(w, rq)


def test_batch_beyond_the_default_shared_memory_size():
    """5000 requests: the verify kernel's per-request tables exceed 48 KB of shared memory."""
    w = small(V=11, k_cap=2)
    rng = np.random.default_rng(13)
    hists = [rng.integers(0, 3, int(n)) for n in rng.integers(0, 40, 5000)]
    rq = hand_requests(w, hists, rng.integers(0, 3, 5000))
    run(w, rq)


def test_two_calls_with_different_shapes_share_a_context():
    """A context sized for the larger call serves a smaller one afterwards (scratch at rest)."""
    w = small()
    rng = np.random.default_rng(11)
    big = hand_requests(w, [rng.integers(0, 4, 5000) for _ in range(20)], [8] * 20)
    sm = hand_requests(w, [rng.integers(0, 4, 100) for _ in range(3)], [8] * 3)
    ctx = G.make_ctx(w, big)
    for rq in (big, sm, big):
        inp = P.prepare(w.scaled(B=rq.B), device="cuda", rq=rq.copy())
        G.run_and_compare(inp, ctx=ctx)
    ctx.close()


def test_host_side_argument_errors():
    import paper_2606_01019_b200 as H
    w = small()
    rng = np.random.default_rng(12)
    rq = hand_requests(w, [rng.integers(0, 4, 100) for _ in range(3)], [8] * 3)
    ctx = G.make_ctx(w, rq)
    b = G.make_batch(ctx, w, rq)
    with pytest.raises(H.HvdError, match="hvd_set_predictor first"):
        b.score_select()
    with pytest.raises(H.HvdError, match="B outside"):
        ctx.hvd_lookup(4, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.K, b.n_max, b.draft, b.draft_len,
                       b.match_len, b.match_pos, b.match_cnt)
    with pytest.raises(H.HvdError, match="NULL"):
        ctx.hvd_lookup(3, None, b.hist_off, b.hist_cap, b.hist_len, b.K, b.n_max, b.draft, b.draft_len,
                       b.match_len, b.match_pos, b.match_cnt)
    with pytest.raises(H.HvdError, match="n_max"):
        ctx.hvd_lookup(3, b.hist, b.hist_off, b.hist_cap, b.hist_len, b.K, 10**6, b.draft, b.draft_len,
                       b.match_len, b.match_pos, b.match_cnt)
    assert ctx.hvd_device_status() == 0
    with pytest.raises(H.HvdError):
        H.Context(max_batch=0, k_cap=8, max_hist_len=10, max_rows=10, max_vocab=10)
    with pytest.raises(H.HvdError):
        H.Context(max_batch=4, k_cap=65, max_hist_len=10, max_rows=10, max_vocab=10)
    with pytest.raises(H.HvdError):
        H.Context(max_batch=4, k_cap=8, max_hist_len=2**31 - 1, max_rows=10, max_vocab=10)
    ctx.close()


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("B,n_top", [(60, 50000), (20, 100000), (33, 100000), (10, 200000), (40, 100000)])
def test_long_histories_in_small_batches(B, n_top, fused):
    """The lookup shapes for histories beyond 32 K tokens: a request's chunks as one thread-block cluster of 8 or 16
    CTAs of 256 threads (60 x 50 000, 20 x 100 000), of 8 or 16 CTAs of 512 threads (33 x 100 000, 10 x 200 000), or
    as plain CTAs that meet through global memory when the clusters do not all fit at once (40 x 100 000).  Ragged
    on purpose: one request of full length, the others anywhere below it (empty chunks inside a cluster), lengths
    at the chunk edges, slabs off the 16-byte grid, unusable lengths, and a small vocabulary so that every warp
    has candidates to extend."""
    w = small(V=211)
    rng = np.random.default_rng(1000 * B + n_top // 1000)
    lens = [n_top, 0, 1, 2, 8192, 8193, 8195, 16384, 16385, 32768, 32769, 32772, n_top - 1, n_top - 3]
    lens = [min(x, n_top) for x in lens][:B]
    lens += [int(x) for x in rng.integers(3, n_top + 1, B - len(lens))]
    hists = []
    for i, n in enumerate(lens):
        h = rng.integers(0, 3 if i % 3 else w.V, n)
        if n > 200 and i % 2 == 0:               # a long match planted somewhere inside, in whatever chunk
            t = int(rng.integers(2, 100))
            e0 = int(rng.integers(t, n - t))
            h[e0 - t:e0] = h[n - t:]
        hists.append(h)
    hist_len = list(lens)
    hist_len[5], hist_len[6] = -7, 2**31 - 1     # unusable lengths: skipped with neutral outputs
    mis = [i % 4 for i in range(B)]
    rq = hand_requests(w, hists, [int(k) for k in rng.integers(0, 9, B)], hist_len=hist_len, misalign=mis)
    (g, out, _), _ = run(w, rq, fused=fused)
    assert (out.lk.match_len >= 2).sum() >= (B - 5) // 2   # five requests are empty, too short or unusable


def test_history_of_more_than_65535_chunks():
    """A history so long that its chunks outgrow the y range of a grid (the launch then puts the chunks
    on x): 537 M tokens in one request, the longest match planted far inside."""
    import torch
    w = small(k_cap=16)
    n = 65536 * 8192 + 4321
    rng = np.random.default_rng(21)
    h = rng.integers(0, 1 << 30, n, dtype=np.int32)
    tail = h[n - 24:].copy()
    h[400_000_000:400_000_024] = tail            # the copy the lookup has to find, in a far chunk
    h[123_456_789 - 9:123_456_789] = tail[-9:]   # a shorter one
    rq = hand_requests(w, [h], [16])
    del h
    lk = P.lookup(w, rq, nthreads=1)
    assert lk.match_len[0] == 24 and lk.match_pos[0] == 400_000_024 and lk.draft_len[0] == 16
    ctx = G.make_ctx(w, rq)
    b = G.make_batch(ctx, w, rq)
    b.lookup()
    torch.cuda.synchronize()
    assert ctx.hvd_device_status() == 0
    got = dict(draft=b.draft, draft_len=b.draft_len, match_len=b.match_len, match_pos=b.match_pos,
               match_cnt=b.match_cnt)
    G.compare_lookup({k: v.cpu().numpy() for k, v in got.items()}, lk)
    ctx.close()


def test_parity_with_plain_launches():
    """The same parity cases with programmatic dependent launch switched off (every kernel starts after
    its predecessor has completed): a result must not depend on how far consecutive kernels overlap."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, HVD_PDL_MASK="0")
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "tests/test_gpu_parity.py", "tests/test_gpu_prefix.py",
           "-k", "c1_full or fused_lookup or multi_step or chained or switching or scaled_workloads or every_accepted"]
    res = subprocess.run(cmd, cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout


def _rerun(env_over, files, select):
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", *files, "-k", select]
    res = subprocess.run(cmd, cwd=root, env=dict(os.environ, **env_over), capture_output=True, text=True, timeout=1200)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout


def test_parity_with_the_persistent_streaming_kernel_only():
    """Logits of up to 160 MB are streamed by the warp-per-batch kernels, so most cases of this suite never
    reach the persistent kernel: the shape, alignment, tie and multi-step cases once more with the limit at 0."""
    _rerun({"HVD_VERIFY_SMALL_BYTES": "0"}, ["tests/test_gpu_parity.py", "tests/test_gpu_edge_cases.py"],
           "not full_size and not plain_launches and not kernel_only and not 65535 and not chunk_lookup_only and not bounds_checked")


def test_parity_with_the_warp_per_batch_kernel_on_a_large_call():
    """... and the other way round: the full-size C2 and C5 workloads (279 MB and 2.5 GB of logits, uniform and
    ragged rows) through the warp-per-batch kernel that checks the need first."""
    _rerun({"HVD_VERIFY_SMALL_BYTES": str(1 << 40)}, ["tests/test_gpu_parity.py"], "full_size and (C2 or C5)")


def test_parity_with_the_chunk_lookup_only():
    """Batches of long histories that fit the GPU in one wave take the cluster form of the lookup (a request's chunk
    CTAs as one thread-block cluster); the same cases once more with the plain chunk kernel and its global
    combine, which larger batches use."""
    _rerun({"HVD_LOOKUP_CLUSTER": "0"}, ["tests/test_gpu_parity.py", "tests/test_gpu_random_sweep.py"],
           "(full_size and C4) or random_batches")


def test_edge_cases_against_the_bounds_checked_build():
    """The stand-in for a memory checker: the library built with -DHVD_DEBUG_BOUNDS tests every index of the
    lookup, commit and streaming kernels before the access and records a violation in the device status word.
    The edge, shape and random cases once more against that build (with both streaming kernels); every context
    must close with status 0, and the results must still equal the oracle's."""
    from paper_2606_01019_b200 import build
    lib = build.build_bounds_checked()
    sel = "not plain_launches and not kernel_only and not large_call and not bounds_checked and not full_size and not chunk_lookup_only"
    files = ["tests/test_gpu_edge_cases.py", "tests/test_gpu_parity.py", "tests/test_gpu_cycle.py", "tests/test_gpu_tree.py",
             "tests/test_gpu_random_sweep.py", "tests/test_gpu_prefix.py"]
    _rerun({"HVD_B200_LIB": lib, "HVD_ASSERT_DEVICE_STATUS": "1"}, files, sel)
    _rerun({"HVD_B200_LIB": lib, "HVD_ASSERT_DEVICE_STATUS": "1", "HVD_VERIFY_SMALL_BYTES": "0"},
           ["tests/test_gpu_edge_cases.py"], sel)
