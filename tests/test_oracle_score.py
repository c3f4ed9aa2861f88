"""Pins for the oracle's payoff features, MLP score and threshold rule (Sec. 3.3, Sec. 3.4)."""
import numpy as np
import torch

import hvd_workloads as W
from oracle import hvd_oracle as O
from oracle import pipeline as P


def f32(x):
    return np.float32(x)


def test_feature_closed_forms():
    # all recent steps selected the cache, every recent accepted length 8
    phi = O.features_one(1000, 250, 0xFF, 0x0808080808080808, 5, 12, 900, 3)
    assert phi[0] == 12 and phi[1] == 5
    assert phi[2] == 2                       # bit width of 3
    assert phi[3] == f32(100) / f32(1000)    # recency (n - pos) / n
    assert phi[4] == 8                       # bit width of 250
    assert phi[5] == f32(750) / f32(1000)
    assert phi[6] == 1.0 and phi[7] == 8.0
    # nothing selected, nothing accepted, no match, empty history
    phi = O.features_one(0, 0, 0, 0, 0, 0, -1, 0)
    assert (phi == 0).all()
    # only the low 8 selection bits count; ring bytes are summed individually
    phi = O.features_one(64, 64, 0xFFFFFF01, 0x00000000000000FF, 1, 2, 1, 1)
    assert phi[6] == f32(1) / f32(8) and phi[7] == f32(255) / f32(8)
    assert phi[2] == 1 and phi[3] == f32(63) / f32(64) and phi[4] == 7 and phi[5] == 0.0


def test_features_match_numpy_float32():
    rng = np.random.default_rng(5)
    for _ in range(500):
        n = int(rng.integers(1, 200000)); Pn = int(rng.integers(0, n + 1))
        L = int(rng.integers(0, 65)); d = int(rng.integers(0, L + 1)) if L else 0
        pos = int(rng.integers(1, n)) if (L and n > 1) else -1
        cnt = int(rng.integers(1, 5000)) if L else 0
        sb = int(rng.integers(0, 2**32)); ring = int(rng.integers(0, 2**63))
        phi = O.features_one(n, Pn, sb, ring, d, L, pos, cnt)
        want = np.array([L, d, cnt.bit_length(),
                         0 if pos < 0 else f32(n - pos) / f32(n),
                         Pn.bit_length(), f32(n - Pn) / f32(n),
                         f32(bin(sb & 0xFF).count("1")) / f32(8),
                         f32(sum((ring >> (8 * j)) & 0xFF for j in range(8))) / f32(8)], np.float32)
        assert (phi == want).all()


def test_mlp_closed_forms():
    H, F = 32, 8
    phi = np.arange(1, 9, dtype=np.float32) * f32(0.37)
    Z1, zb, Z2 = np.zeros((H, F), np.float32), np.zeros(H, np.float32), np.zeros(H, np.float32)
    assert O.mlp_f32(phi, Z1, zb, Z2, 2.5) == 2.5                       # zero weights: y = b2
    for k in range(F):
        for j in (0, 13, 31):
            W1 = Z1.copy(); W1[j, k] = 1.0
            W2 = Z2.copy(); W2[j] = 1.0
            b1 = zb.copy(); b1[j] = 0.25
            assert O.mlp_f32(phi, W1, b1, W2, 1.0) == f32(1.0) + (phi[k] + f32(0.25))
            b1[j] = -100.0                                               # negative pre-activation: ReLU kills it
            assert O.mlp_f32(phi, W1, b1, W2, 1.0) == 1.0
            W1[j, k] = -1.0; b1[j] = 0.0
            assert O.mlp_f32(phi, W1, b1, W2, 1.0) == 1.0
    # a transposed W1 would give a different answer on a non-symmetric case
    W1 = Z1.copy(); W1[3, 5] = 2.0
    W2 = Z2.copy(); W2[3] = 0.5
    assert O.mlp_f32(phi, W1, zb, W2, 0.0) == f32(0.5) * (f32(2.0) * phi[5])


def test_mlp_against_fp64_and_torch():
    rng = np.random.default_rng(11)
    for H in (32, 7, 256):
        W1 = rng.normal(0, 0.1, (H, 8)).astype(np.float32); b1 = rng.normal(0, 0.1, H).astype(np.float32)
        W2 = rng.normal(0, 0.1, H).astype(np.float32)
        for _ in range(50):
            phi = np.abs(rng.normal(0, 10, 8)).astype(np.float32)
            y32 = O.mlp_f32(phi, W1, b1, W2, 6.0)
            y64 = O.mlp_f64(phi, W1, b1, W2, 6.0)
            t = torch.nn.functional.linear(
                torch.relu(torch.nn.functional.linear(torch.from_numpy(phi).double(),
                                                      torch.from_numpy(W1).double(),
                                                      torch.from_numpy(b1).double())),
                torch.from_numpy(W2).double()[None], torch.tensor([6.0]).double())
            assert abs(y64 - float(t)) <= 1e-12 * max(1.0, abs(y64))
            assert abs(y32 - y64) <= 1e-5 * max(1.0, abs(y64))


def _score(B, draft_len, W1, b1, W2, b2, tau, model_len=None, K=None, k_cap=4):
    lk = O.LookupOut(np.tile(np.arange(10, 10 + k_cap, dtype=np.int32), (B, 1)), np.asarray(draft_len, np.int32),
                     np.asarray(draft_len, np.int32), np.full(B, 5, np.int32), np.ones(B, np.int32))
    for b in range(B):
        lk.draft[b, draft_len[b]:] = -1
    st = np.zeros(B, O.STATE_DTYPE)
    md = np.tile(np.arange(100, 100 + k_cap, dtype=np.int32), (B, 1))
    ml = np.full(B, k_cap, np.int32) if model_len is None else np.asarray(model_len, np.int32)
    K = np.full(B, k_cap, np.int32) if K is None else np.asarray(K, np.int32)
    return O.score_select(np.full(B, 50, np.int32), np.full(B, 20, np.int32), st, K, lk, md, ml,
                          k_cap=k_cap, W1=W1, b1=b1, W2=W2, b2=b2, tau=tau)


def test_threshold_rule():
    Z1, zb, Z2 = np.zeros((32, 8), np.float32), np.zeros(32, np.float32), np.zeros(32, np.float32)
    # score == tau exactly -> cache (the rule is >=); no cache draft -> model whatever the score
    out = _score(3, [3, 0, 4], Z1, zb, Z2, 6.0, 6.0)
    assert list(out.select) == [1, 0, 1] and (out.score == 6.0).all()
    assert list(out.sel_len) == [3, 4, 4]
    assert list(out.sel_draft[0]) == [10, 11, 12, -1] and list(out.sel_draft[1]) == [100, 101, 102, 103]
    below = float(np.nextafter(np.float32(6.0), np.float32(0.0)))
    out = _score(2, [3, 4], Z1, zb, Z2, below, 6.0)
    assert list(out.select) == [0, 0] and list(out.sel_len) == [4, 4]
    # model draft is clamped to the request's K; a missing model draft gives an empty draft
    out = _score(2, [0, 0], Z1, zb, Z2, 0.0, 6.0, model_len=[9, 3], K=[2, 4])
    assert list(out.sel_len) == [2, 3] and list(out.sel_draft[0]) == [100, 101, -1, -1]


def test_scores_on_workload_fp32_vs_fp64():
    w = W.CONFIGS["C2"].scaled(B=32, n=2048)
    rq = W.make_requests(w)
    W1, b1, W2, b2, tau = W.make_predictor(w)
    lk = P.lookup(w, rq)
    sc = P.score_select(w, rq, lk, W1, b1, W2, b2, tau)
    assert np.abs(sc.score - sc.score64).max() <= 1e-5 * np.abs(sc.score64).max()
    assert ((sc.select == 1) == ((lk.draft_len > 0) & (sc.score >= np.float32(tau)))).all()
    assert (sc.sel_len[sc.select == 1] == lk.draft_len[sc.select == 1]).all()
    assert (sc.sel_len[sc.select == 0] == rq.model_len[sc.select == 0]).all()


# ---- two hidden layers: the paper's predictor shape (App. B: 2 hidden layers, ReLU) -------------------
def test_mlp2_closed_forms():
    H, F = 16, 8
    phi = np.arange(1, 9, dtype=np.float32) * f32(0.25)
    Z1, z, ZH = np.zeros((H, F), np.float32), np.zeros(H, np.float32), np.zeros((H, H), np.float32)
    assert O.mlp2_f32(phi, Z1, z, ZH, z, z, 3.5) == 3.5                       # all zero: y = output bias
    # a single path phi_k -> h1[a] -> h2[c] -> y with unit weights: y = b + relu(relu(phi_k + b1) + bh)
    for k, a, c in [(0, 0, 0), (5, 3, 11), (7, 15, 2)]:
        W1 = Z1.copy(); W1[a, k] = 1.0
        Wh = ZH.copy(); Wh[c, a] = 1.0                                            # row c reads h1[a]
        W2 = z.copy(); W2[c] = 1.0
        b1 = z.copy(); b1[a] = 0.5
        bh = z.copy(); bh[c] = 0.125
        assert O.mlp2_f32(phi, W1, b1, Wh, bh, W2, 1.0) == f32(1.0) + ((phi[k] + f32(0.5)) + f32(0.125))
        if a != c:                                                                # a transposed Wh breaks the path:
            Wt = ZH.copy(); Wt[a, c] = 1.0                                        # only relu(bh[c]) reaches the output
            assert O.mlp2_f32(phi, W1, b1, Wt, bh, W2, 1.0) == f32(1.0) + f32(0.125)
        bh[c] = -100.0                                                            # second ReLU cuts the path
        assert O.mlp2_f32(phi, W1, b1, Wh, bh, W2, 1.0) == 1.0
        bh[c] = 0.125; b1[a] = -100.0                                             # first ReLU cuts it: only bh is left
        assert O.mlp2_f32(phi, W1, b1, Wh, bh, W2, 1.0) == f32(1.0) + f32(0.125)
    # an identity second layer reduces the network to the one-layer predictor
    W1 = np.random.default_rng(1).normal(0, 0.1, (H, F)).astype(np.float32)
    b1 = np.random.default_rng(2).normal(0, 0.1, H).astype(np.float32)
    W2 = np.random.default_rng(3).normal(0, 0.1, H).astype(np.float32)
    assert O.mlp2_f32(phi, W1, b1, np.eye(H, dtype=np.float32), z, W2, 2.0) == O.mlp_f32(phi, W1, b1, W2, 2.0)


def test_mlp2_against_fp64_and_torch():
    rng = np.random.default_rng(12)
    for H in (8, 64, 256):
        W1 = rng.normal(0, 0.1, (H, 8)).astype(np.float32); b1 = rng.normal(0, 0.1, H).astype(np.float32)
        Wh = rng.normal(0, 0.1, (H, H)).astype(np.float32); bh = rng.normal(0, 0.1, H).astype(np.float32)
        W2 = rng.normal(0, 0.1, H).astype(np.float32)
        for _ in range(20):
            phi = np.abs(rng.normal(0, 10, 8)).astype(np.float32)
            y32 = O.mlp2_f32(phi, W1, b1, Wh, bh, W2, 6.0)
            y64 = O.mlp2_f64(phi, W1, b1, Wh, bh, W2, 6.0)
            lin = torch.nn.functional.linear
            d = lambda x: torch.from_numpy(x).double()
            t = lin(torch.relu(lin(torch.relu(lin(d(phi), d(W1), d(b1))), d(Wh), d(bh))), d(W2)[None],
                    torch.tensor([6.0]).double())
            assert abs(y64 - float(t)) <= 1e-12 * max(1.0, abs(y64))
            assert abs(y32 - y64) <= 2e-5 * max(1.0, abs(y64))


def test_two_layer_scores_on_workload():
    w = W.CONFIGS["C2"].scaled(B=32, n=2048, hidden=256, hidden_layers=2)
    inp = P.prepare(w)
    out = P.step(inp, inp.rq.copy())
    sc = out.sc
    assert inp.Wh.shape == (256, 256)
    assert np.abs(sc.score - sc.score64).max() <= 2e-5 * np.abs(sc.score64).max()
    assert 0 < sc.select.sum() < len(sc.select)
    for b in range(4):
        assert sc.score[b] == np.float32(O.mlp2_f32(sc.features[b], inp.W1, inp.b1, inp.Wh, inp.bh, inp.W2, inp.b2))
