#!/usr/bin/env python
"""Measurements of the variants of the HVD path (the rows the scope marks "next"): trace-replay labels,
frequency-weighted lookup, shared warm-up corpus, vocabulary shards.  Each prints ONE JSON line.

    python bench_variants.py --replay | --freq | --corpus | --vocab-shards [--config C2] [--steps K] [--warmup W]

The headline benchmark of the per-step path is bench.py; nothing here is part of its timed region.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 2**20


# ----------------------------------------------------------------------------------------------
# second workload: trace-replay labels (training-data path)
# ----------------------------------------------------------------------------------------------
def run_replay(args):
    import torch
    import hvd_workloads as W
    import paper_2606_01019_b200 as H
    torch.cuda.set_device(0)
    w = W.CONFIGS[args.config]
    rq = W.make_requests(w.scaled(B=min(w.B, 4)))
    x = np.ascontiguousarray(rq.history(0), np.int32)
    n, K = len(x), int(rq.K[0])
    ctx = H.Context(max_batch=4096, k_cap=w.k_cap, max_hist_len=n, max_rows=1, max_vocab=1, l_max=w.l_max,
                    min_match=w.min_match)
    xd = torch.as_tensor(x, device="cuda")
    outs = [torch.zeros(n, dtype=torch.int32, device="cuda") for _ in range(5)]
    for _ in range(max(3, args.warmup)):
        ctx.hvd_replay_labels(xd, n, K, *outs)
    torch.cuda.synchronize()
    reps = max(1, min(args.steps, 50))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        ctx.hvd_replay_labels(xd, n, K, *outs)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    label = outs[0].cpu().numpy()
    from oracle import hvd_oracle as O
    from oracle import pipeline as P
    cores = P.host_threads()
    t0 = time.perf_counter()
    ref = O.replay_labels(x, K, k_cap=w.k_cap, l_max=w.l_max, min_match=w.min_match, nthreads=cores)
    cpu_s = time.perf_counter() - t0
    line = {"metric": "trace-replay labelled positions/s", "value": n / (ms * 1e-3), "unit": "positions/s",
            "n_gpus": 1, "steps": reps, "ms_per_trace": ms, "higher_is_better": True, "dtype": "int32",
            "data": "synthetic", "config": {"workload": f"replay of one {w.name} history: {n} positions, K {K}",
                                            "launches_per_trace": 2},
            "prefix_tokens_scanned_per_trace": int(n) * (int(n) + 1) // 2,
            "scan_rate_gtokens_per_s": int(n) * (int(n) + 1) / 2 / (ms * 1e-3) / 1e9,
            "mean_label": float(label.mean()), "labels_ge_6_frac": float((label >= 6).mean()),
            "cpu_baseline": {"value": n / cpu_s, "unit": "positions/s", "cores": cores, "kind": "oracle",
                             "sample": "the same whole trace, once", "agrees_with_gpu": bool((ref.label == label).all())}}
    print(json.dumps(line), flush=True)
    ctx.close()


# ----------------------------------------------------------------------------------------------
# variant of the lookup step: frequency-weighted draft and suffix score
# ----------------------------------------------------------------------------------------------
def run_freq(args):
    import torch
    import hvd_workloads as W
    import paper_2606_01019_b200 as H
    torch.cuda.set_device(0)
    w = W.CONFIGS[args.config]
    rq = W.make_requests(w)
    B, n_max = rq.B, int(rq.hist_len.max())
    dev = lambda a: torch.as_tensor(np.ascontiguousarray(a), device="cuda")
    hist, off, cap, ln, K = dev(rq.hist), dev(rq.hist_off), dev(rq.hist_cap), dev(rq.hist_len), dev(rq.K)
    i32 = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda")
    draft, dlen, mlen, mpos, mcnt = i32(B, w.k_cap), i32(B), i32(B), i32(B), i32(B)
    score = torch.zeros(B, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    from oracle import hvd_oracle as O
    from oracle import pipeline as P
    cores = P.host_threads()
    reps = max(3, min(args.steps, 50))
    cases = []
    for l_max in (w.l_max, 2):   # the configured maximum match length, and a short one (many occurrences per request)
        ctx = H.Context(max_batch=B, k_cap=w.k_cap, max_hist_len=int(rq.hist_cap.max()), max_rows=1, max_vocab=1,
                        l_max=l_max, min_match=min(w.min_match, l_max), spec_factor=8.0)
        calls = {"hvd_lookup": lambda: ctx.hvd_lookup(B, hist, off, cap, ln, K, n_max, draft, dlen, mlen, mpos, mcnt),
                 "hvd_lookup_freq": lambda: ctx.hvd_lookup_freq(B, hist, off, cap, ln, K, n_max, 0.1, H.FREQ_MAX_OCC, 0.0,
                                                                None, None, draft, dlen, score, mlen, mpos, mcnt)}
        us = {}
        for name, call in calls.items():
            for _ in range(max(3, args.warmup)):
                call()
            evs = []
            for _ in range(reps):   # all enqueued ahead: the fills hide the host's launch latency
                flush.fill_(1)      # L2 flush between timed calls
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); call(); e1.record()
                evs.append((e0, e1))
            torch.cuda.synchronize()
            us[name] = sum(a.elapsed_time(b) for a, b in evs) / reps * 1e3
        t0 = time.perf_counter()
        ref = O.lookup_freq(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, k_cap=w.k_cap, l_max=l_max,
                            min_match=min(w.min_match, l_max), spec_factor=8.0, min_prob=0.1, max_occ=H.FREQ_MAX_OCC,
                            nthreads=cores)
        cpu_s = time.perf_counter() - t0
        agrees = bool((ref.draft == draft.cpu().numpy()).all() and
                      (ref.score.view(np.uint32) == score.cpu().numpy().view(np.uint32)).all())
        cases.append({"l_max": l_max, "us_lookup": us["hvd_lookup"], "us_lookup_freq": us["hvd_lookup_freq"],
                      "mean_occurrences": float(ref.match_cnt.mean()), "max_occurrences": int(ref.match_cnt.max()),
                      "merged_requests": int(((ref.match_cnt > 0) & (ref.match_cnt <= H.FREQ_MAX_OCC)).sum()),
                      "mean_draft_len": float(ref.draft_len.mean()), "mean_score": float(ref.score.mean()),
                      "oracle_ms": cpu_s * 1e3, "agrees_with_oracle": agrees})
        ctx.close()
    hist_bytes = int(rq.hist_len.sum()) * 4
    c0 = cases[0]
    line = {"metric": "frequency-weighted lookups/s", "value": B / (c0["us_lookup_freq"] * 1e-6), "unit": "requests/s",
            "n_gpus": 1, "steps": reps, "higher_is_better": True, "dtype": "int32 (fp32 score)", "data": "synthetic",
            "config": {"workload": f"{w.name}: batch {B}, histories {w.n} tokens; 3 launches per call, "
                                   "L2 flushed between calls", "history_bytes": hist_bytes},
            "history_scan_gbs": 2 * hist_bytes / (c0["us_lookup_freq"] * 1e-6) / 1e9,
            "cases": cases,
            "cpu_baseline": {"value": B / (c0["oracle_ms"] * 1e-3), "unit": "requests/s", "cores": cores, "kind": "oracle",
                             "sample": "the same batch, once"}}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# variant of the lookup step: shared warm-up corpus
# ----------------------------------------------------------------------------------------------
def run_corpus(args):
    import torch
    import hvd_workloads as W
    import paper_2606_01019_b200 as H
    torch.cuda.set_device(0)
    w = W.CONFIGS[args.config]
    rq = W.make_requests(w)
    B, n_max = rq.B, int(rq.hist_len.max())
    dev = lambda a: torch.as_tensor(np.ascontiguousarray(a), device="cuda")
    hist, off, cap, ln, K = dev(rq.hist), dev(rq.hist_off), dev(rq.hist_cap), dev(rq.hist_len), dev(rq.K)
    i32 = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda")
    draft, dlen, mlen, mpos, msrc, mcnt = i32(B, w.k_cap), i32(B), i32(B), i32(B), i32(B), i32(B)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    from oracle import hvd_oracle as O
    from oracle import pipeline as P
    cores = P.host_threads()
    reps = max(3, min(args.steps, 50))
    ctx = H.Context(max_batch=B, k_cap=w.k_cap, max_hist_len=int(rq.hist_cap.max()), max_rows=1, max_vocab=1,
                    l_max=w.l_max, min_match=w.min_match)

    def timed(call, cold):
        for _ in range(max(3, args.warmup)):
            call()
        evs = []
        for _ in range(reps):   # all enqueued ahead: the fills hide the host's launch latency
            if cold:
                flush.fill_(1)  # L2 flush between timed calls
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); call(); e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in evs) / reps * 1e3

    plain = lambda: ctx.hvd_lookup(B, hist, off, cap, ln, K, n_max, draft, dlen, mlen, mpos, mcnt)
    both = lambda: ctx.hvd_lookup_corpus(B, hist, off, cap, ln, K, n_max, draft, dlen, mlen, mpos, msrc, mcnt)
    us_plain = timed(plain, True)
    cases = []
    for n_traces in (16, 64, 256):
        corpus = W.make_corpus(w, n_traces=n_traces)
        cd = dev(corpus)
        ctx.hvd_set_corpus(cd)
        us_cold, us_warm = timed(both, True), timed(both, False)
        t0 = time.perf_counter()
        ref = O.lookup_corpus(rq.hist, rq.hist_off, rq.hist_cap, rq.hist_len, rq.K, corpus, k_cap=w.k_cap,
                              l_max=w.l_max, min_match=w.min_match, nthreads=cores)
        cpu_s = time.perf_counter() - t0
        agrees = all(bool((getattr(ref, k) == t.cpu().numpy()).all()) for k, t in
                     (("draft", draft), ("draft_len", dlen), ("match_len", mlen), ("match_pos", mpos),
                      ("match_src", msrc), ("match_cnt", mcnt)))
        m = len(corpus)
        cases.append({"corpus_tokens": m, "us_lookup_corpus_cold": us_cold, "us_lookup_corpus_corpus_in_l2": us_warm,
                      "token_compares_per_s": float(B) * m / (us_warm * 1e-6),
                      "requests_matched_in_corpus": int(ref.match_src.sum()), "oracle_ms": cpu_s * 1e3,
                      "agrees_with_oracle": agrees})
    c = cases[1]
    line = {"metric": "lookups over corpus and history per second", "value": B / (c["us_lookup_corpus_cold"] * 1e-6),
            "unit": "requests/s", "n_gpus": 1, "steps": reps, "higher_is_better": True, "dtype": "int32",
            "data": "synthetic",
            "config": {"workload": f"{w.name}: batch {B}, histories {w.n} tokens, warm-up corpus of {c['corpus_tokens']} "
                                   "tokens (64 traces); 2 launches per call, L2 flushed between calls"},
            "us_lookup_history_only": us_plain, "cases": cases,
            "cpu_baseline": {"value": B / (c["oracle_ms"] * 1e-3), "unit": "requests/s", "cores": cores, "kind": "oracle",
                             "sample": "the same batch and corpus, once"}}
    print(json.dumps(line), flush=True)
    ctx.close()


# ----------------------------------------------------------------------------------------------
# variant of the verify step: vocabulary shards (one rank's work; the 8-bytes-per-row MAX all-reduce
# between the two calls needs the other ranks and is not part of this single-GPU timing)
# ----------------------------------------------------------------------------------------------
def run_vocab_shards(args):
    import torch
    import hvd_workloads as W
    import paper_2606_01019_b200 as H
    from paper_2606_01019_b200.runner import DeviceBatch
    torch.cuda.set_device(0)
    w = W.CONFIGS[args.config]
    # inputs as in the main arm: the selection comes from the CUDA path itself, the logits are planted on it
    rq = W.make_requests(w)
    W1, b1, W2, b2, tau = W.make_predictor(w)
    B, rows = rq.B, int(rq.row_off[-1])
    ctx = H.Context(max_batch=B, k_cap=w.k_cap, max_hist_len=int(rq.hist_cap.max()), max_rows=rows, max_vocab=w.V,
                    l_max=w.l_max, min_match=w.min_match, hidden=w.hidden)
    ctx.hvd_set_predictor(W1, b1, W2, b2, tau)
    batch = DeviceBatch(ctx, hist=rq.hist, hist_off=rq.hist_off, hist_cap=rq.hist_cap, hist_len=rq.hist_len, K=rq.K,
                        prompt_len=rq.prompt_len, state=rq.state, model_draft=rq.model_draft, model_len=rq.model_len,
                        row_off=rq.row_off, V=w.V, dtype=w.dtype)
    batch.lookup_score_select()
    if w.calibrate_cache_frac is not None:
        torch.cuda.synchronize()
        tau = W.calibrate_tau(batch.score.cpu().numpy(), batch.draft_len.cpu().numpy() > 0, w.calibrate_cache_frac)
        ctx.hvd_set_predictor(W1, b1, W2, b2, tau)
        batch.lookup_score_select()
    torch.cuda.synchronize()
    sel_len_h, sel_draft_h = batch.sel_len.cpu().numpy(), batch.sel_draft.cpu().numpy()
    logits = W.make_logits(w, rows, device="cuda")
    W.plant_agreement(w, logits, rq.row_off, sel_draft_h, sel_len_h, W.make_agreement(w, sel_len_h))
    full = logits.reshape(-1)[: rows * w.V].reshape(rows, w.V)
    needed = int((batch.sel_len.cpu().numpy().astype(np.int64) + 1).sum())
    hist_len0, state0 = batch.hist_len.clone(), batch.state.clone()
    reps = max(3, min(args.steps, 50))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    cases = []
    for S in (1, 2, 4, 8):
        Vs = w.V // S
        copies = [full[:, :Vs].contiguous() for _ in range(2 if S > 1 else 1)]
        keys = torch.zeros(rows, dtype=torch.int64, device="cuda")

        def call(i):
            ctx.hvd_verify_keys(B, copies[i % len(copies)], batch.dtype, Vs, 0, batch.row_off, 0, rows, batch.sel_len,
                                batch.hist_len, batch.hist_cap, keys)
            ctx.hvd_commit_keys(B, keys, w.V, batch.row_off, 0, rows, batch.sel_draft, batch.sel_len, batch.select,
                                batch.hist, batch.hist_off, batch.hist_cap, batch.hist_len, batch.state, batch.accepted,
                                batch.committed, batch.n_commit, None, batch.status)

        def body(i, with_call):
            batch.hist_len.copy_(hist_len0); batch.state.copy_(state0)
            flush.fill_(1)   # L2 flush between calls
            if with_call:
                call(i)

        for i in range(3):
            body(i, True)
        torch.cuda.synchronize()
        stream = torch.cuda.Stream()
        times = []
        for with_call in (True, False):   # the same graph with and without the calls: the difference is the calls
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(stream):
                g.capture_begin()
                for i in range(reps):
                    body(i, with_call)
                g.capture_end()
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                g.replay()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); g.replay(); e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        us = (times[0] - times[1]) / reps * 1e3
        shard_bytes = needed * Vs * w.elt
        cases.append({"shards": S, "us_per_rank": us, "shard_bytes": shard_bytes, "gbs": shard_bytes / (us * 1e-6) / 1e9,
                      "allreduce_bytes_per_rank": rows * 8, "logits_allgather_bytes_avoided": needed * (w.V - Vs) * w.elt})
    line = {"metric": "verify+commit per rank under vocabulary shards", "value": cases[-1]["us_per_rank"], "unit": "us",
            "n_gpus": 1, "steps": reps, "higher_is_better": False, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": f"{w.name}: batch {B}, {rows} logits rows, vocab {w.V} in S slices; one rank's "
                                   "hvd_verify_keys + hvd_commit_keys (4 kernels) in a CUDA graph, L2 flushed between calls; "
                                   "time = graph with the calls minus the same graph without them"},
            "cases": cases}
    print(json.dumps(line), flush=True)
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="C2")
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    g = ap.add_mutually_exclusive_group(required=True)
    g.add_argument("--replay", action="store_true", help="payoff labels by trace replay (hvd_replay_labels) on one history of the config")
    g.add_argument("--freq", action="store_true", help="frequency-weighted draft and score (hvd_lookup_freq) on the config's requests")
    g.add_argument("--corpus", action="store_true", help="shared warm-up corpus scanned with the history (hvd_lookup_corpus)")
    g.add_argument("--vocab-shards", action="store_true",
                   help="one rank's share under a vocabulary-parallel output layer (hvd_verify_keys + hvd_commit_keys), S = 1, 2, 4, 8")
    args = ap.parse_args()
    if args.replay:
        run_replay(args)
    elif args.freq:
        run_freq(args)
    elif args.corpus:
        run_corpus(args)
    else:
        run_vocab_shards(args)


if __name__ == "__main__":
    main()
