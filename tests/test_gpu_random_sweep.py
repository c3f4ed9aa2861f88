"""GPU parity on randomly drawn batches: batch size, draft cap, vocabulary size, logits type, hidden width,
history content and length, slab alignment, free space and invalid lengths all vary together; every case runs
one of the three call sequences (separate calls, fused lookup + scoring, commit fused with the next lookup)
and is compared with the oracle array by array."""
import numpy as np
import pytest

import hvd_workloads as W
from oracle import pipeline as P
from tests import gpu_helpers as G
from tests.test_gpu_cycle import run_chain
from tests.test_gpu_edge_cases import hand_requests

pytestmark = pytest.mark.gpu

LENGTHS = [0, 1, 2, 3, 5, 17, 100, 1023, 1024, 1025, 2047, 4096, 5000, 9000, 16384, 20000, 33000]


def draw_case(rng, it):
    B = int(rng.integers(1, 41))
    kc = int(rng.choice([1, 4, 8, 16, 31, 32, 33, 64]))
    V = int(rng.choice([1, 2, 7, 33, 997, 4099, 32003, 50257]))
    w = W.CONFIGS["C2"].scaled(B=B, V=V, k_cap=kc, K=kc, dtype=str(rng.choice(["bf16", "f32"])),
                               hidden=int(rng.choice([1, 8, 32, 64])),
                               calibrate_cache_frac=float(rng.uniform(0.1, 0.9)))
    tv = max(1, min(int(rng.choice([2, 3, 5, 50, 1000])), V))      # token values in the histories
    base = rng.integers(0, tv, 40000)
    hists, Ks, extra, mis = [], [], [], []
    for _ in range(B):
        kind = int(rng.integers(0, 4))
        n = int(rng.choice(LENGTHS)) if kind == 0 else int(rng.integers(0, 6000))
        if kind == 1:
            h = base[:n]                                            # shared prefix: long matches
        elif kind == 2:
            h = rng.integers(0, tv, n)
        else:
            h = np.resize(rng.integers(0, tv, max(1, int(rng.integers(1, 40)))), n)   # periodic
        hists.append(h)
        Ks.append(int(rng.integers(0, kc + 1)))
        extra.append(int(rng.choice([0, 1, 2, kc, 4 * (kc + 1), 10 * (kc + 1)])))
        mis.append(int(rng.integers(0, 4)))
    lens = [len(h) for h in hists]
    if rng.random() < 0.3:                                          # a length outside its slab
        j = int(rng.integers(0, B))
        lens[j] = int(rng.choice([-1, len(hists[j]) + extra[j] + 1]))
    rq = hand_requests(w, hists, Ks, cap_extra=extra, hist_len=lens, misalign=mis, seed=it)
    return w.scaled(B=B), rq


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_batches(seed):
    for it in range(60):
        rng = np.random.default_rng(seed * 100000 + it)
        w, rq = draw_case(rng, it)
        inp = P.prepare(w, device="cuda", rq=rq)
        mode = int(rng.integers(0, 3))
        try:
            if mode == 0:
                run_chain(inp, rq, 3)
            else:
                G.run_and_compare(inp, fused=(mode == 1), rq=rq.copy())
        except AssertionError as e:
            raise AssertionError(f"seed {seed} case {it} (B {w.B}, k_cap {w.k_cap}, V {w.V}, {w.dtype}, mode {mode}): {e}")


LONG = [9000, 16385, 20000, 32768, 32769, 33000, 40000, 65536, 65540, 100000, 131072, 200000, 262144, 300000]


def draw_long_case(rng, it):
    """Batches around one long history: the lookup shapes beyond 8 K tokens (one CTA of 1024 threads per request,
    512 threads x 16 loads, chunk CTAs that meet through global memory, clusters of 4 to 16 chunk CTAs)."""
    n_top = int(rng.choice(LONG))
    B = int(rng.integers(1, 80)) if n_top <= 70000 else int(rng.integers(1, 40))
    kc = int(rng.choice([1, 8, 16, 32, 64]))
    V = int(rng.choice([2, 7, 997, 32003]))
    w = W.CONFIGS["C2"].scaled(B=B, V=V, k_cap=kc, K=kc, dtype=str(rng.choice(["bf16", "f32"])), hidden=32,
                               calibrate_cache_frac=float(rng.uniform(0.1, 0.9)))
    tv = max(1, min(int(rng.choice([2, 3, 50, 1000, 30000])), V))
    hists, Ks, extra, mis = [], [], [], []
    for b in range(B):
        kind = int(rng.integers(0, 4))
        if b == 0:
            n = n_top
        elif kind:
            n = int(rng.integers(0, n_top + 1))
        else:
            n = min(int(rng.choice([0, 1, 2, 8192, 8195, 16384, 32768, 32771, n_top - 1])), n_top)
        if kind == 3:
            h = np.resize(rng.integers(0, tv, max(1, int(rng.integers(1, 90)))), n)          # periodic
        else:
            h = rng.integers(0, tv, n)
            if n > 300 and kind == 2:                                                        # a planted copy of the tail
                t = int(rng.integers(2, 120))
                e0 = int(rng.integers(t, n - t))
                h[e0 - t:e0] = h[n - t:]
        hists.append(h)
        Ks.append(int(rng.integers(0, kc + 1)))
        extra.append(int(rng.choice([0, 1, kc, 4 * (kc + 1), 10 * (kc + 1), 5000])))
        mis.append(int(rng.integers(0, 4)))
    lens = [len(h) for h in hists]
    if rng.random() < 0.3:
        j = int(rng.integers(0, B))
        lens[j] = int(rng.choice([-1, len(hists[j]) + extra[j] + 1]))
    rq = hand_requests(w, hists, Ks, cap_extra=extra, hist_len=lens, misalign=mis, seed=it)
    return w.scaled(B=B), rq


@pytest.mark.parametrize("seed", [21, 22])
def test_random_batches_of_long_histories(seed):
    for it in range(40):
        rng = np.random.default_rng(seed * 100000 + it)
        w, rq = draw_long_case(rng, it)
        inp = P.prepare(w, device="cuda", rq=rq)
        mode = int(rng.integers(0, 3))
        try:
            if mode == 0:
                run_chain(inp, rq, 3)
            else:
                G.run_and_compare(inp, fused=(mode == 1), rq=rq.copy())
        except AssertionError as e:
            raise AssertionError(f"seed {seed} case {it} (B {w.B}, k_cap {w.k_cap}, V {w.V}, {w.dtype}, mode {mode}): {e}")

