"""Pins for the oracle's greedy verification and commit (Sec. 3.1, Sec. 3.4, Algorithm 1)."""
import os

import numpy as np
import pytest
import torch

import hvd_workloads as W
from oracle import hvd_oracle as O
from oracle import pipeline as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x):
    return torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("V", [1, 7, 8, 9, 1000, 32000])
def test_argmax_equals_library_first_maximum(V):
    rng = np.random.default_rng(V)
    for _ in range(20):
        x = rng.normal(0, 2, V).astype(np.float32)
        assert O.argmax_row(x, O.F32) == int(np.argmax(x))
        xb = bf16_bits(x)                       # coarse grid: ties at the maximum do occur
        wide = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).float()
        assert O.argmax_row(xb, O.BF16) == int(torch.argmax(wide)) == int(np.argmax(wide.numpy()))


def test_argmax_constructed_ties():
    V = 1000
    x = np.zeros(V, np.float32)
    assert O.argmax_row(x, O.F32) == 0                          # all equal
    x[:] = -1.0; x[700] = 3.0; x[20] = 3.0
    assert O.argmax_row(x, O.F32) == 20                         # duplicate maximum: lower index
    x[:] = -0.0; x[5] = 0.0
    assert O.argmax_row(x, O.F32) == 0                          # -0.0 == +0.0
    x[:] = -5.0; x[999] = np.inf; x[998] = np.inf
    assert O.argmax_row(x, O.F32) == 998
    x[:] = -np.inf
    assert O.argmax_row(x, O.F32) == 0
    x[:] = -5.0; x[999] = -4.0
    assert O.argmax_row(x, O.F32) == 999                        # maximum in the last slot
    xb = bf16_bits(np.full(V, -1.0)); xb[3] = 0x8000; xb[9] = 0x0000   # -0.0 then +0.0
    assert O.argmax_row(xb, O.BF16) == 3


def run_verify(draft, targets, V=50, cap_extra=10, n0=5, select=1, dtype=O.F32, k_cap=None):
    """One request whose logits rows have their strict maximum at `targets`."""
    m = len(draft)
    k_cap = k_cap or max(m, 1)
    rows = len(targets)
    logits = np.random.default_rng(0).normal(0, 1, (rows, V)).astype(np.float32)
    for i, t in enumerate(targets):
        logits[i, t] = 20.0
    if dtype == O.BF16:
        logits = bf16_bits(logits)
    hist = np.full(n0 + cap_extra, -7, np.int32); hist[:n0] = np.arange(n0) + 40
    hist_len = np.array([n0], np.int32)
    state = np.zeros(1, O.STATE_DTYPE); state["sel_bits"] = 0b1011; state["acc_ring"] = 0x0102
    sd = np.full((1, k_cap), -1, np.int32); sd[0, :m] = draft
    out = O.verify_commit(logits, dtype, V, np.array([0, rows], np.int64), 0, sd, [m], [select], k_cap=k_cap,
                          hist=hist, hist_off=[0], hist_cap=[n0 + cap_extra], hist_len=hist_len, state=state)
    return out, hist, hist_len, state


@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_hand_worked_fixture(dtype):
    for line in open(os.path.join(GOLDEN, "accepted_length_cases.txt")):
        line = line.split("#")[0].rstrip("\n")
        if not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        draft = [int(x) for x in f[0].split()]; targets = [int(x) for x in f[1].split()]
        a = int(f[2]); z = [int(x) for x in f[3].split()]
        out, hist, hist_len, state = run_verify(draft, targets, dtype=dtype, k_cap=4)
        assert out.accepted[0] == a and out.n_commit[0] == a + 1, line
        assert list(out.committed[0, :a + 1]) == z and (out.committed[0, a + 1:] == -1).all(), line
        assert list(hist[5:5 + a + 1]) == z and hist_len[0] == 5 + a + 1
        assert (hist[:5] == np.arange(5) + 40).all() and (hist[5 + a + 1:] == -7).all()
        assert list(out.target_tok[:len(draft) + 1]) == targets[:len(draft) + 1]
        assert state["sel_bits"][0] == (0b1011 << 1 | 1) and state["acc_ring"][0] == (0x0102 << 8 | a)
        assert out.status[0] == O.REQ_OK


def test_capacity_clamp_and_bad_len():
    out, hist, hist_len, state = run_verify([5, 7, 9], [5, 7, 9, 4], cap_extra=4)     # exactly a+1 free
    assert out.status[0] == O.REQ_OK and out.n_commit[0] == 4
    out, hist, hist_len, state = run_verify([5, 7, 9], [5, 7, 9, 4], cap_extra=3)     # a free slots
    assert out.status[0] == O.REQ_CAPACITY and out.n_commit[0] == 3 and out.accepted[0] == 3
    assert list(hist[5:8]) == [5, 7, 9] and hist_len[0] == 8
    assert list(out.committed[0]) == [5, 7, 9, 4]
    out, hist, hist_len, state = run_verify([5, 7, 9], [5, 7, 9, 4], cap_extra=0)
    assert out.status[0] == O.REQ_CAPACITY and out.n_commit[0] == 0 and hist_len[0] == 5
    # unusable length: nothing happens
    logits = np.zeros((2, 10), np.float32)
    hist = np.arange(8, dtype=np.int32); hl = np.array([9], np.int32); st = np.zeros(1, O.STATE_DTYPE)
    out = O.verify_commit(logits, O.F32, 10, None, 1, np.zeros((1, 1), np.int32), [1], [1], k_cap=1,
                          hist=hist, hist_off=[0], hist_cap=[8], hist_len=hl, state=st)
    assert out.status[0] == O.REQ_BAD_LEN and out.n_commit[0] == 0 and hl[0] == 9
    assert (hist == np.arange(8)).all() and st["sel_bits"][0] == 0


def test_rows_after_the_rejection_are_not_counted():
    # row 1 rejects; rows 2 and 3 would agree again
    out, *_ = run_verify([5, 7, 9, 11], [5, 1, 9, 11, 2], k_cap=4)
    assert out.accepted[0] == 1 and list(out.committed[0, :2]) == [5, 1]
    assert list(out.target_tok) == [5, 1, 9, 11, 2]


def test_out_of_vocab_draft_never_matches():
    out, *_ = run_verify([-1, 7], [5, 7, 9], k_cap=2)
    assert out.accepted[0] == 0 and out.committed[0, 0] == 5
    out, *_ = run_verify([50, 7], [5, 7, 9], V=50, k_cap=2)
    assert out.accepted[0] == 0


@pytest.mark.parametrize("name", ["C1", "C2"])
def test_workload_commit_equals_plain_greedy_decoding(name):
    w = W.CONFIGS[name]
    if name == "C2":
        w = w.scaled(B=16, n=4096, V=20011)        # odd vocabulary: rows are not 16-byte multiples
    inp = P.prepare(w)
    rq = inp.rq.copy()
    out = P.step(inp, rq, nthreads=4)
    vf, sc = out.vf, out.sc
    if w.dtype == "bf16":
        wide = torch.from_numpy(inp.logits_np.view(np.int16)).view(torch.bfloat16).float().numpy()
    else:
        wide = inp.logits_np
    wide = wide.reshape(-1, w.V)
    for b in range(rq.B):
        r0, m, a = int(rq.row_off[b]), int(sc.sel_len[b]), int(vf.accepted[b])
        assert 0 <= a <= m <= rq.K[b]
        # every committed token is its row's greedy token (library argmax): plain greedy decoding
        for j in range(a + 1):
            assert vf.committed[b, j] == int(np.argmax(wide[r0 + j]))
        # label equation of Sec. 3.3 evaluated with the library argmax
        t = [int(np.argmax(wide[r0 + i])) for i in range(m + 1)]
        y = max(l for l in range(m + 1) if list(sc.sel_draft[b, :l]) == t[:l])
        assert a == y
        assert list(vf.target_tok[r0:r0 + m + 1]) == t
        assert (vf.target_tok[r0 + m + 1:int(rq.row_off[b + 1])] == -1).all()
        # history grew by exactly the committed block; everything before is untouched
        n0 = int(inp.rq.hist_len[b])
        assert rq.hist_len[b] == n0 + a + 1 and vf.n_commit[b] == a + 1
        assert (rq.slab(b)[:n0] == inp.rq.slab(b)[:n0]).all()
        assert (rq.slab(b)[n0:n0 + a + 1] == vf.committed[b, :a + 1]).all()
        assert (rq.slab(b)[n0 + a + 1:] == W.FREE_VALUE).all()
        assert rq.state["sel_bits"][b] == ((int(inp.rq.state["sel_bits"][b]) << 1) | int(sc.select[b])) & 0xFFFFFFFF
        assert rq.state["acc_ring"][b] == ((int(inp.rq.state["acc_ring"][b]) << 8) | a) & (2**64 - 1)
    assert (vf.accepted == inp.A)[inp.strict].all()          # planted prefix is recovered exactly
    assert (rq.hist[rq.guard_mask] == W.GUARD_VALUE).all()   # canaries intact
    assert (vf.status == O.REQ_OK).all()
    assert sc.select.sum() > 0 and (sc.select == 0).sum() > 0


def test_multi_step_loop_keeps_appending():
    w = W.CONFIGS["C1"]
    inp = P.prepare(w)
    rq = inp.rq.copy()
    total = np.zeros(rq.B, np.int64)
    for s in range(4):
        logits = W.make_logits(w, int(rq.row_off[-1]), salt=100 + s)
        out = P.step(inp, rq, logits_np=W.logits_to_numpy(logits))
        total += out.vf.n_commit
        assert (out.vf.status == O.REQ_OK).all()
    assert (rq.hist_len == inp.rq.hist_len + total).all() and (total >= 4).all()
    assert (rq.hist[rq.guard_mask] == W.GUARD_VALUE).all()


# ---- token-tree drafts (the paper's model drafter proposes trees: App. A drafting configuration) --------
def run_tree(draft, parent, targets, V=50, k_cap=None, n0=5, cap_extra=12):
    m = len(draft)
    k_cap = k_cap or max(m, 1)
    rows = len(targets)
    logits = np.random.default_rng(1).normal(0, 1, (rows, V)).astype(np.float32)
    for i, t in enumerate(targets):
        logits[i, t] = 20.0
    hist = np.full(n0 + cap_extra, -7, np.int32); hist[:n0] = np.arange(n0) + 40
    hist_len = np.array([n0], np.int32)
    state = np.zeros(1, O.STATE_DTYPE)
    sd = np.full((1, k_cap), -1, np.int32); sd[0, :m] = draft
    par = np.full((1, k_cap), -9, np.int32); par[0, :m] = parent
    out = O.verify_commit(logits, O.F32, V, np.array([0, rows], np.int64), 0, sd, [m], [0], k_cap=k_cap, hist=hist,
                          hist_off=[0], hist_cap=[n0 + cap_extra], hist_len=hist_len, state=state, parent=par)
    return out, hist, hist_len


def test_tree_hand_worked():
    #            prefix
    #          /        \
    #      n0:5          n1:6
    #     /    \           \
    #  n2:7    n3:8        n4:9
    #            \
    #            n5:3
    draft, parent = [5, 6, 7, 8, 9, 3], [-1, -1, 0, 0, 1, 3]
    # rows: 0 after the prefix, i+1 after node i.  Target says 5, then (after n0) 8, then (after n3) 3,
    # then (after n5) 4: path n0 n3 n5 accepted, bonus 4.
    targets = [5, 8, 1, 1, 3, 1, 4]
    out, hist, hl = run_tree(draft, parent, targets)
    assert out.accepted[0] == 3 and list(out.committed[0, :4]) == [5, 8, 3, 4] and hl[0] == 9
    assert list(hist[5:9]) == [5, 8, 3, 4]
    # the target prefers 6 at the root and then something no child of n1 carries: one accepted, bonus 2
    out, *_ = run_tree(draft, parent, [6, 1, 2, 1, 1, 1, 1])
    assert out.accepted[0] == 1 and list(out.committed[0, :2]) == [6, 2]
    # the target's first token is nobody's: nothing accepted
    out, *_ = run_tree(draft, parent, [4, 8, 9, 1, 3, 1, 1])
    assert out.accepted[0] == 0 and out.committed[0, 0] == 4
    # siblings with the same token: the first one is taken (and its subtree decides what follows)
    out, *_ = run_tree([5, 5, 7, 8], [-1, -1, 0, 1], [5, 8, 7, 1, 1])
    assert out.accepted[0] == 1 and list(out.committed[0, :2]) == [5, 8]


def test_tree_chain_equals_linear_verification():
    rng = np.random.default_rng(31)
    for _ in range(50):
        m = int(rng.integers(0, 9))
        draft = list(rng.integers(0, 6, m))
        targets = list(rng.integers(0, 6, m + 1))
        a, h1, l1, _ = run_verify(draft, targets, V=50, k_cap=8)
        b, h2, l2 = run_tree(draft, list(range(-1, m - 1)), targets, V=50, k_cap=8)
        assert a.accepted[0] == b.accepted[0] and (a.committed == b.committed).all() and l1[0] == l2[0]


def test_tree_against_path_enumeration():
    """Brute force: among all root paths, the accepted one is the path whose every token equals the
    target's token at its parent and that cannot be extended; children are tried in index order."""
    rng = np.random.default_rng(32)
    for _ in range(300):
        m = int(rng.integers(1, 12))
        parent = [int(rng.integers(-1, i)) for i in range(m)]
        draft = [int(x) for x in rng.integers(0, 4, m)]
        targets = [int(x) for x in rng.integers(0, 4, m + 1)]
        cur, path = -1, []
        while True:
            kids = [c for c in range(m) if parent[c] == cur and draft[c] == targets[cur + 1]]
            if not kids:
                break
            cur = kids[0]
            path.append(draft[cur])
        out, *_ = run_tree(draft, parent, targets, V=10, k_cap=12)
        assert out.accepted[0] == len(path)
        assert list(out.committed[0, :len(path) + 1]) == path + [targets[cur + 1]]
