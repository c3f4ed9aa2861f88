"""Whole-step driver around the CPU oracle (test infrastructure only).

`prepare` draws one seeded input set for a workload and plants the logits so that they agree with
the drafts THE ORACLE selects; `step` runs lookup -> score/select -> verify/commit on host arrays.
Nothing here is used by the CUDA package.
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import numpy as np

import hvd_workloads as W
from oracle import hvd_oracle as O


def host_threads() -> int:
    return len(os.sched_getaffinity(0))


@dataclass
class Inputs:
    w: W.Workload
    rq: W.Requests          # pristine requests (copy before stepping)
    W1: np.ndarray
    b1: np.ndarray
    W2: np.ndarray
    b2: float
    tau: float
    Wh: object = None       # second hidden layer [H,H] (None: one-layer predictor)
    bh: object = None
    A: np.ndarray = None    # planted accepted lengths
    strict: np.ndarray = None      # requests on which accepted == A must hold
    logits: object = None          # torch tensor [rows, V] on the device it was drawn on
    logits_np: np.ndarray = None   # host copy (float32, or uint16 bf16 bit patterns)


@dataclass
class StepOut:
    lk: O.LookupOut
    sc: O.ScoreOut
    vf: O.VerifyOut


def lookup(w, rq, nthreads=1):
    return O.lookup(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, k_cap=w.k_cap,
                    l_max=w.l_max, min_match=w.min_match, nthreads=nthreads)


def score_select(w, rq, lk, W1, b1, W2, b2, tau, nthreads=1, Wh=None, bh=None):
    return O.score_select(rq.hist_len, rq.prompt_len, rq.state, rq.K, lk, rq.model_draft, rq.model_len,
                          k_cap=w.k_cap, W1=W1, b1=b1, W2=W2, b2=b2, tau=tau, nthreads=nthreads, Wh=Wh, bh=bh)


def verify_commit(w, rq, sc, logits_np, nthreads=1):
    dtype = O.F32 if w.dtype == "f32" else O.BF16
    return O.verify_commit(logits_np, dtype, w.V, rq.row_off, 0, sc.sel_draft, sc.sel_len, sc.select,
                           k_cap=w.k_cap, hist=rq.hist, hist_off=rq.hist_off, hist_cap=rq.hist_cap,
                           hist_len=rq.hist_len, state=rq.state, nthreads=nthreads)


def prepare(w: W.Workload, device="cpu", nthreads=None, salt: int = 0, rq: W.Requests = None) -> Inputs:
    """Seeded inputs for one step.  `rq` replaces the generated requests (hand-built edge cases)."""
    nthreads = nthreads or host_threads()
    rq = W.make_requests(w) if rq is None else rq
    W1, b1, W2, b2, tau = W.make_predictor(w)
    Wh, bh = W.make_second_layer(w) if w.hidden_layers == 2 else (None, None)
    lk = lookup(w, rq, nthreads)
    sc = score_select(w, rq, lk, W1, b1, W2, b2, tau, nthreads, Wh, bh)
    if w.calibrate_cache_frac is not None:
        tau = W.calibrate_tau(sc.score, lk.draft_len > 0, w.calibrate_cache_frac)
        sc = score_select(w, rq, lk, W1, b1, W2, b2, tau, nthreads, Wh, bh)
    A = W.make_agreement(w, sc.sel_len)
    logits = W.make_logits(w, max(int(rq.row_off[-1]), 1), device=device, salt=salt)
    strict = W.plant_agreement(w, logits, rq.row_off, sc.sel_draft, sc.sel_len, A, salt=salt)
    return Inputs(w, rq, W1, b1, W2, b2, tau, Wh, bh, A, strict, logits, W.logits_to_numpy(logits))


def step(inp: Inputs, rq: W.Requests, nthreads=1, logits_np=None) -> StepOut:
    """One decoding step on `rq` (updated in place: history, lengths, state)."""
    w = inp.w
    lk = lookup(w, rq, nthreads)
    sc = score_select(w, rq, lk, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, nthreads, inp.Wh, inp.bh)
    vf = verify_commit(w, rq, sc, inp.logits_np if logits_np is None else logits_np, nthreads)
    return StepOut(lk, sc, vf)
