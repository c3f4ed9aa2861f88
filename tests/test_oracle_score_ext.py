"""Pins for the oracle's extended feature vector (App. B feature groups: the draft-structure group and
the suffix score) and for scoring on it."""
import numpy as np
import torch

import hvd_workloads as W
from oracle import hvd_oracle as O

f32 = np.float32


def test_hand_worked_class_shares():
    cls = np.zeros(100, np.uint8)
    cls[5] = 0b00001; cls[6] = 0b10110; cls[7] = 0b00011
    phi = O.features_ext_one(1000, 250, 0xFF, 0x0808080808080808, [5, 6, 7, 99, 100, -1], 12, 900, 3, cls, 2.5)
    base = O.features_one(1000, 250, 0xFF, 0x0808080808080808, 6, 12, 900, 3)
    assert (phi[:8] == base).all()
    # whitespace: tokens 5 and 7; punctuation: 6 and 7; line break: 6; bracket: none; delimiter: 6;
    # tokens 100 and -1 lie outside the table and carry no class
    assert list(phi[8:13]) == [f32(2) / f32(6), f32(2) / f32(6), f32(1) / f32(6), f32(0), f32(1) / f32(6)]
    assert phi[13] == f32(2.5)
    # empty draft: no shares, no division
    phi = O.features_ext_one(10, 2, 0, 0, [], 0, -1, 0, cls)
    assert (phi[8:] == 0).all()
    # every token in every class
    phi = O.features_ext_one(10, 2, 0, 0, [1, 1, 1], 3, 4, 1, np.full(4, 0xFF, np.uint8))
    assert (phi[8:13] == 1).all()


def test_class_shares_match_numpy():
    rng = np.random.default_rng(12)
    for _ in range(400):
        V = int(rng.integers(1, 300))
        cls = rng.integers(0, 256, V).astype(np.uint8)
        d = int(rng.integers(0, 65))
        draft = rng.integers(-2, V + 3, d).astype(np.int32)
        phi = O.features_ext_one(500, 100, 1, 2, draft, 5, 17, 2, cls, 0.0)
        ok = (draft >= 0) & (draft < V)
        bits = np.unpackbits(cls[draft[ok]][:, None], axis=1, bitorder="little")[:, :5] if ok.any() else np.zeros((0, 5))
        want = [f32(bits[:, k].sum()) / f32(d) if d else f32(0) for k in range(5)]
        assert list(phi[8:13]) == want


def test_mlp_on_fourteen_features_against_fp64_and_torch():
    rng = np.random.default_rng(2)
    for H in (1, 7, 64, 256):
        W1 = rng.normal(0, 0.5, (H, 14)).astype(f32); b1 = rng.normal(0, 0.5, H).astype(f32)
        W2 = rng.normal(0, 0.5, H).astype(f32); b2 = 0.25
        phi = rng.uniform(0, 16, 14).astype(f32)
        y32, y64 = O.mlp_f32(phi, W1, b1, W2, b2), O.mlp_f64(phi, W1, b1, W2, b2)
        t = lambda a: torch.tensor(a, dtype=torch.float64)
        ref = float(t(W2) @ torch.relu(t(W1) @ t(phi) + t(b1)) + b2)
        assert abs(y64 - ref) <= 1e-12 * max(1.0, abs(ref))
        mag = float(np.abs(W2).astype(np.float64) @ (np.abs(W1).astype(np.float64) @ phi + np.abs(b1)) + abs(b2))
        assert abs(y32 - ref) <= 4 * (H + 16) * 2.0**-24 * mag
    # a transposed or shifted first layer would change this closed form: one unit reading feature 9 only
    W1 = np.zeros((1, 14), f32); W1[0, 9] = 3.0
    phi = np.arange(14, dtype=f32)
    assert O.mlp_f32(phi, W1, [0.5], [2.0], 1.0) == 2.0 * (3.0 * 9 + 0.5) + 1.0


def _inputs(B=40, k_cap=16, V=5000, seed=4):
    rng = np.random.default_rng(seed)
    w = W.CONFIGS["C2"].scaled(B=B, n=3000, V=V)
    rq = W.make_requests(w)
    lk = O.lookup(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, k_cap=w.k_cap, nthreads=4)
    cls = rng.integers(0, 32, V).astype(np.uint8)
    sfx = rng.uniform(0, 16, B).astype(f32)
    return w, rq, lk, cls, sfx


def test_zero_weights_on_the_new_features_give_the_base_score():
    w, rq, lk, cls, sfx = _inputs()
    W1, b1, W2, b2, _ = W.make_predictor(w)
    W1x = np.concatenate([W1, np.zeros((W1.shape[0], 6), f32)], axis=1)
    args = (rq.hist_len, rq.prompt_len, rq.state, rq.K, lk)
    base = O.score_select(*args, rq.model_draft, rq.model_len, k_cap=w.k_cap, W1=W1, b1=b1, W2=W2, b2=b2, tau=6.0)
    ext = O.score_select_ext(*args, sfx, cls, rq.model_draft, rq.model_len, k_cap=w.k_cap, W1=W1x, b1=b1, W2=W2, b2=b2,
                             tau=6.0)
    assert (ext.score.view(np.uint32) == base.score.view(np.uint32)).all()
    assert (ext.features[:, :8] == base.features).all()
    assert (ext.select == base.select).all() and (ext.sel_draft == base.sel_draft).all()
    assert (ext.features[:, 13] == sfx).all()
    # and with a second layer
    Wh, bh = W.make_second_layer(w)
    base2 = O.score_select(*args, rq.model_draft, rq.model_len, k_cap=w.k_cap, W1=W1, b1=b1, W2=W2, b2=b2, tau=6.0, Wh=Wh, bh=bh)
    ext2 = O.score_select_ext(*args, sfx, cls, rq.model_draft, rq.model_len, k_cap=w.k_cap, W1=W1x, b1=b1, W2=W2, b2=b2,
                              tau=6.0, Wh=Wh, bh=bh)
    assert (ext2.score.view(np.uint32) == base2.score.view(np.uint32)).all()


def test_single_feature_probes():
    """One hidden unit reading one new feature: the score is that feature times the weight."""
    w, rq, lk, cls, sfx = _inputs()
    args = (rq.hist_len, rq.prompt_len, rq.state, rq.K, lk)
    for i in range(8, 14):
        W1 = np.zeros((1, 14), f32); W1[0, i] = 2.0
        out = O.score_select_ext(*args, sfx, cls, None, None, k_cap=w.k_cap, W1=W1, b1=[0.0], W2=[1.0], b2=0.0, tau=0.5)
        assert (out.score == f32(2.0) * out.features[:, i]).all()
        if i < 13:
            for b in range(rq.B):
                d = lk.draft[b, :lk.draft_len[b]]
                want = f32(((cls[d] >> (i - 8)) & 1).sum()) / f32(len(d)) if len(d) else f32(0)
                assert out.features[b, i] == want
        assert (out.select == ((lk.draft_len > 0) & (out.score >= f32(0.5)))).all()
    none = O.score_select_ext(*args, None, cls, None, None, k_cap=w.k_cap, W1=np.zeros((1, 14), f32), b1=[0.0], W2=[1.0],
                              b2=0.0, tau=0.5)
    assert (none.features[:, 13] == 0).all()


def test_corpus_matches_take_position_zero():
    w, rq, lk, cls, sfx = _inputs()
    args = (rq.hist_len, rq.prompt_len, rq.state, rq.K, lk)
    kw = dict(k_cap=w.k_cap, W1=np.zeros((1, 14), f32), b1=[0.0], W2=[1.0], b2=0.0, tau=0.5)
    src = (np.arange(rq.B) % 2).astype(np.int32)
    a = O.score_select_ext(*args, sfx, cls, None, None, **kw)
    b = O.score_select_ext(*args, sfx, cls, None, None, match_src=src, **kw)
    has = lk.match_len > 0
    assert (b.features[(src == 1) & has, 3] == 1.0).all()            # (n - 0) / n
    assert (b.features[src == 0] == a.features[src == 0]).all()
    cols = [i for i in range(14) if i != 3]
    assert (b.features[:, cols] == a.features[:, cols]).all()
