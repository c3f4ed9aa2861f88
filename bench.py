#!/usr/bin/env python
"""Benchmark of the HVD per-step path (lookup -> score/select -> verify/commit) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C2] [--impl b200|reference]

One step = one pass of the whole path over one batch of seeded synthetic input.  Prints ONE JSON
line.  With N > 1 (launched by torch.distributed.run) every rank runs its own copy of the batch:
requests are independent, so the path shards with no collective on the data path ("weak" scaling);
only the timing is reduced (max over ranks).

Timed region: K steps captured in one CUDA graph (3 kernel launches per step), bracketed by a
barrier + synchronize, timed with CUDA events on the launching stream.  Consecutive steps use
rotating copies of the big inputs (histories, logits) so that nothing a step reads is left in L2
by an earlier step, and every step gets pristine per-step lengths/state.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "HVD select+verify steps/s"
UNIT = "steps/s"
L2_BYTES = 126 * 2**20
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one verify_commit launch on this workload, from
# the ncu capture summarised under profiles/ (None until captured for a workload)
NCU_VERIFY_TRAFFIC_BYTES = {"C2": 261772928}  # profiles/verify_stream_kernel_c2_ncu.txt, mean of two launches


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="C2")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--mode", default="graph", choices=["graph", "stream"])
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--predictor", default="config", choices=["config", "2x256"],
                    help="2x256: the paper's predictor shape (two hidden layers of 256 units) instead of the config's")
    ap.add_argument("--freq", action="store_true",
                    help="variant of the lookup step: frequency-weighted draft and score (hvd_lookup_freq) on the config's requests")
    ap.add_argument("--corpus", action="store_true",
                    help="variant of the lookup step: shared warm-up corpus scanned with the history (hvd_lookup_corpus)")
    ap.add_argument("--vocab-shards", action="store_true",
                    help="variant of the verify step: one rank's share under a vocabulary-parallel output layer "
                         "(hvd_verify_keys on a 1/S slice of every row + hvd_commit_keys), S = 2, 4, 8")
    ap.add_argument("--verify-sweep", action="store_true",
                    help="the verify call over batch sizes 1..64 (C2's rows), with both streaming kernels")
    ap.add_argument("--replay", action="store_true",
                    help="second workload: payoff labels by trace replay (hvd_replay_labels) on one history of the config")
    ap.add_argument("--unfused", action="store_true",
                    help="call hvd_lookup and hvd_score_select separately instead of hvd_lookup_score_select")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="leave the per-kernel event records out of the timed graph")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------------
# clocks during the timed region
# ----------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
               0x100: "display_clock_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # pragma: no cover
            self.err = repr(e)

    def sample(self):
        nv = self.nv
        mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
        except Exception:
            bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
        self.samples.append(mhz)
        for bit, name in self.REASONS.items():
            if bits & bit:
                self.reasons.add(name)

    def run(self):
        if not self.ok:
            return
        while not self.stop_flag.is_set():
            try:
                self.sample()
            except Exception:
                break
            time.sleep(self.period)

    def summary(self, window: str):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "window": window}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples), "window": window}


# ----------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ----------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import hvd_workloads as W
    from oracle import pipeline as P
    w = W.CONFIGS[args.config]
    cores = P.host_threads()
    inp = P.prepare(w, device="cpu", nthreads=cores)
    # one full step to size the per-step sample
    rq = inp.rq.copy()
    t0 = time.perf_counter()
    P.step(inp, rq, nthreads=cores)
    t_full = time.perf_counter() - t0
    budget = 150.0
    B_s = w.B
    if (args.steps + args.warmup) * t_full > budget:
        B_s = max(1, int(w.B * budget / ((args.steps + args.warmup) * t_full)))
    sub = inp
    if B_s < w.B:
        # a bounded sample: the first B_s requests of the batch (own history slabs, own logits rows)
        rows = int(inp.rq.row_off[B_s])
        keep = slice(0, B_s)
        sub = P.Inputs(w, W.subset_requests(inp.rq, 0, B_s), inp.W1, inp.b1, inp.W2, inp.b2, inp.tau,
                       Wh=inp.Wh, bh=inp.bh, A=inp.A[keep], strict=inp.strict[keep], logits=inp.logits[:rows],
                       logits_np=inp.logits_np[:rows])
    times, committed = [], 0
    for i in range(args.warmup + args.steps):
        rq = sub.rq.copy()
        t0 = time.perf_counter()
        out = P.step(sub, rq, nthreads=cores)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
            committed += int(out.vf.n_commit.sum())
    total = float(np.sum(times))
    frac = B_s / w.B
    value = args.steps * frac / total
    sample = (f"{B_s} of {w.B} requests of {w.name} per step (whole-batch-equivalent steps/s = sampled "
              f"steps/s x {frac:.4f})" if B_s < w.B else f"the whole {w.name} batch every step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps / frac,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic", "config": workload_config(w, args.gpus),
            "tokens_per_s": committed / total,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


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


# ----------------------------------------------------------------------------------------------
# the verify call from one request to a full batch: which streaming kernel serves which size
# ----------------------------------------------------------------------------------------------
def run_verify_sweep(args):
    """hvd_verify_commit on 1..64 requests with C2's logits rows (K + 1 = 17 rows of 128 256 bf16 per request),
    selected draft lengths uniform in 0..K (about half the rows needed), timed with the persistent streaming
    kernel only (HVD_VERIFY_SMALL_BYTES=0) and with the library's own choice.  Inputs are random: nothing is
    checked here (the parity tests do that), only timed."""
    import torch
    import hvd_workloads as W
    import paper_2606_01019_b200 as H
    from paper_2606_01019_b200.runner import DeviceBatch
    torch.cuda.set_device(0)
    reps = max(3, min(args.steps, 40))
    cases = []
    for B in (1, 2, 4, 8, 16, 32, 64):
        w = W.CONFIGS["C2"].scaled(B=B, n=2048)
        rq = W.make_requests(w)
        rows = int(rq.row_off[-1])
        full_bytes = rows * w.V * w.elt
        R = int(max(2, min(40, -(-4 * L2_BYTES // full_bytes))))
        logits = [W.make_logits(w, rows, device="cuda", salt=r) for r in range(R)]
        gen = torch.Generator(device="cuda")
        gen.manual_seed(1000 + B)
        sel_len = torch.randint(0, w.K + 1, (B,), generator=gen, device="cuda", dtype=torch.int32)
        sel_draft = torch.randint(0, w.V, (B, w.k_cap), generator=gen, device="cuda", dtype=torch.int32)
        needed_bytes = int((sel_len.cpu().numpy().astype(np.int64) + 1).sum()) * w.V * w.elt
        us = {}
        for kind, env in (("persistent", "0"), ("default", None)):
            old = os.environ.pop("HVD_VERIFY_SMALL_BYTES", None)
            if env is not None:
                os.environ["HVD_VERIFY_SMALL_BYTES"] = env
            ctx = H.Context(max_batch=B, k_cap=w.k_cap, max_hist_len=int(rq.hist_cap.max()), max_rows=rows,
                            max_vocab=w.V, l_max=w.l_max, min_match=w.min_match, hidden=w.hidden)
            os.environ.pop("HVD_VERIFY_SMALL_BYTES", None)
            if old is not None:
                os.environ["HVD_VERIFY_SMALL_BYTES"] = old
            b = DeviceBatch(ctx, hist=rq.hist, hist_off=rq.hist_off, hist_cap=rq.hist_cap, hist_len=rq.hist_len, K=rq.K,
                            prompt_len=rq.prompt_len, state=rq.state, model_draft=rq.model_draft,
                            model_len=rq.model_len, row_off=rq.row_off, V=w.V, dtype=w.dtype)
            b.sel_len.copy_(sel_len); b.sel_draft.copy_(sel_draft); b.select.zero_()
            hl0, st0 = b.hist_len.clone(), b.state.clone()

            def body(i, with_call):
                b.hist_len.copy_(hl0); b.state.copy_(st0)
                if with_call:
                    b.verify_commit(logits[i % R], target_tok=False)

            for i in range(3):
                body(i, True)
            torch.cuda.synchronize()
            stream = torch.cuda.Stream()
            t = []
            for with_call in (True, False):   # the same graph with and without the call
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
                t.append(e0.elapsed_time(e1))
            us[kind] = (t[0] - t[1]) / reps * 1e3
            ctx.close()
        cases.append({"requests": B, "logits_bytes": full_bytes, "needed_bytes": needed_bytes,
                      "us_persistent_kernel": us["persistent"], "us_library_choice": us["default"],
                      "gbs_library_choice": needed_bytes / (us["default"] * 1e-6) / 1e9})
    line = {"metric": "hvd_verify_commit call over batch sizes", "value": cases[0]["us_library_choice"], "unit": "us",
            "n_gpus": 1, "steps": reps, "higher_is_better": False, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "C2's logits rows (17 rows of 128256 bf16 per request), 1..64 requests, selected draft "
                                   "lengths uniform in 0..16; calls in a CUDA graph on rotating logits copies larger than "
                                   "L2 in total; time = graph with the calls minus the same graph without them"},
            "cases": cases}
    print(json.dumps(line), flush=True)


def workload_config(w, n_gpus, extra=None):
    cfg = {"workload": f"{w.name}: batch {w.B}, histories {w.n} tokens, vocab {w.V}, K {w.K}, {w.dtype} logits",
           "requests_per_gpu": w.B, "parallelism": f"requests sharded over {n_gpus} GPU(s), no collective"}
    if extra:
        cfg.update(extra)
    return cfg


# ----------------------------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.freq:
        run_freq(args)
        return
    if args.corpus:
        run_corpus(args)
        return
    if args.vocab_shards:
        run_vocab_shards(args)
        return
    if args.verify_sweep:
        run_verify_sweep(args)
        return
    if args.replay:
        run_replay(args)
        return

    import torch
    import torch.distributed as dist
    import hvd_workloads as W
    import paper_2606_01019_b200 as H
    from paper_2606_01019_b200.sharding import max_over_ranks

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the HVD path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = W.CONFIGS[args.config]
    if args.predictor == "2x256":
        w = w.scaled(hidden=256, hidden_layers=2)
    K_steps, W_steps = args.steps, args.warmup
    n_slots = K_steps + W_steps
    peak_gbs, peak_kind = measured_peak()

    # ---- inputs: the product path itself produces the drafts the logits are planted on ----------
    rq = W.make_requests(w)
    W1, b1, W2, b2, tau = W.make_predictor(w)
    B, kc = rq.B, w.k_cap
    total_rows = int(rq.row_off[-1])
    ctx = H.Context(max_batch=B, k_cap=kc, max_hist_len=int(rq.hist_cap.max()), max_rows=total_rows,
                    max_vocab=w.V, l_max=w.l_max, min_match=w.min_match, hidden=w.hidden)
    Wh, bh = W.make_second_layer(w) if w.hidden_layers == 2 else (None, None)

    def set_predictor(t):
        if Wh is not None:
            ctx.hvd_set_predictor2(W1, b1, Wh, bh, W2, b2, t)
        else:
            ctx.hvd_set_predictor(W1, b1, W2, b2, t)

    set_predictor(tau)
    up = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a, dt), device=dev)
    hist0 = up(rq.hist, np.int32)
    hist_off, hist_cap, Kt = up(rq.hist_off, np.int64), up(rq.hist_cap, np.int32), up(rq.K, np.int32)
    hist_len0, prompt_len = up(rq.hist_len, np.int32), up(rq.prompt_len, np.int32)
    state0 = torch.as_tensor(rq.state.view(np.int64).reshape(B, 2), device=dev)
    model_draft, model_len = up(rq.model_draft, np.int32), up(rq.model_len, np.int32)
    row_off = up(rq.row_off, np.int64)
    n_max = int(rq.hist_len.max())   # every timed step starts from the pristine lengths
    i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=dev)
    draft, draft_len, match_len, match_pos, match_cnt = i32(B, kc), i32(B), i32(B), i32(B), i32(B)
    score = torch.zeros(B, dtype=torch.float32, device=dev)
    select, sel_draft, sel_len = i32(B), i32(B, kc), i32(B)
    accepted, committed, n_commit, status = i32(B), i32(B, kc + 1), i32(B), i32(B)

    def lookup(hist, hist_len):
        ctx.hvd_lookup(B, hist, hist_off, hist_cap, hist_len, Kt, n_max, draft, draft_len, match_len,
                       match_pos, match_cnt)

    def score_select(hist_len, state):
        ctx.hvd_score_select(B, hist_len, prompt_len, state, Kt, draft, draft_len, match_len, match_pos,
                             match_cnt, model_draft, model_len, None, score, select, sel_draft, sel_len)

    def lookup_score_select(hist, hist_len, state):
        ctx.hvd_lookup_score_select(B, hist, hist_off, hist_cap, hist_len, Kt, n_max, prompt_len, state,
                                    model_draft, model_len, draft, draft_len, match_len, match_pos, match_cnt,
                                    None, score, select, sel_draft, sel_len)

    dtype = H.F32 if w.dtype == "f32" else H.BF16

    def verify(logits, hist, hist_len, state):
        ctx.hvd_verify_commit(B, logits, dtype, w.V, row_off, 0, total_rows, sel_draft, sel_len, select, hist,
                              hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, None, status)

    # the commit and the next cycle's lookup + selection in one call; the next selection goes to arrays of its
    # own, so that every timed step verifies the same (pristine) selection
    select_n, sel_draft_n, sel_len_n = i32(B), i32(B, kc), i32(B)
    n_max_next = min(int(rq.hist_cap.max()), n_max + kc + 1)

    def cycle(logits, hist, hist_len, state):
        ctx.hvd_verify_commit_next(B, logits, dtype, w.V, row_off, 0, total_rows, sel_draft, sel_len, select, hist,
                                   hist_off, hist_cap, hist_len, state, accepted, committed, n_commit, None, status,
                                   K=Kt, n_max=n_max_next, prompt_len=prompt_len, model_draft=model_draft,
                                   model_len=model_len, draft=draft, draft_len=draft_len, match_len=match_len,
                                   match_pos=match_pos, match_cnt=match_cnt, features=None, score=score,
                                   next_select=select_n, next_sel_draft=sel_draft_n, next_sel_len=sel_len_n)

    lookup(hist0, hist_len0)
    score_select(hist_len0, state0)
    if w.calibrate_cache_frac is not None:
        torch.cuda.synchronize()
        tau = W.calibrate_tau(score.cpu().numpy(), draft_len.cpu().numpy() > 0, w.calibrate_cache_frac)
        set_predictor(tau)
        score_select(hist_len0, state0)
    torch.cuda.synchronize()
    sel_len_h = sel_len.cpu().numpy()
    sel_draft_h = sel_draft.cpu().numpy()
    A = W.make_agreement(w, sel_len_h)
    logits0 = W.make_logits(w, total_rows, device=dev)
    W.plant_agreement(w, logits0, rq.row_off, sel_draft_h, sel_len_h, A)

    # ---- rotating copies of the big inputs, pristine per-step small arrays ------------------------
    foot = hist0.numel() * 4 + logits0.numel() * logits0.element_size()
    R = int(max(2, -(-4 * L2_BYTES // foot)))
    hists = [hist0] + [hist0.clone() for _ in range(R - 1)]
    logits = [logits0] + [logits0.clone() for _ in range(R - 1)]
    hist_len_steps = hist_len0.repeat(n_slots, 1).contiguous()
    state_steps = state0.repeat(n_slots, 1, 1).contiguous()
    hist_len_pristine, state_pristine = hist_len_steps.clone(), state_steps.clone()

    def restore():
        hist_len_steps.copy_(hist_len_pristine)
        state_steps.copy_(state_pristine)

    def step(slot, events=None, with_verify=True, lookup_only=False, verify_only=False, probe_only=False,
             cycle_only=False):
        r = slot % R
        hl, st = hist_len_steps[slot], state_steps[slot]
        if cycle_only:    # verify + commit + the next cycle's lookup and selection: two kernels per step
            cycle(logits[r], hists[r], hl, st)
            return
        if probe_only:    # plain read loop over the same logits buffer: the part's read-only speed
            ctx.hvd_read_probe(logits[r], logits[r].numel() * logits[r].element_size())
            return
        if lookup_only:
            lookup(hists[r], hl)
            return
        if verify_only:   # the selection of the last lookup is still in place: every step starts from the same state
            verify(logits[r], hists[r], hl, st)
            return
        if events is not None:
            events[0].record()
        if args.unfused:
            lookup(hists[r], hl)
            score_select(hl, st)
        else:
            lookup_score_select(hists[r], hl, st)
        if events is not None:
            events[1].record()
        if with_verify:
            verify(logits[r], hists[r], hl, st)
        if events is not None:
            events[2].record()

    # ---- warm-up (eager), then the timed K steps --------------------------------------------------
    for s in range(W_steps):
        step(s)
    torch.cuda.synchronize()
    mode = args.mode
    stream = torch.cuda.Stream(device=dev)

    def capture(events=None, with_verify=True, lookup_only=False, verify_only=False, probe_only=False,
                cycle_only=False):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            g.capture_begin()
            for s in range(K_steps):
                step(W_steps + s, events[s] if events else None, with_verify, lookup_only, verify_only, probe_only,
                     cycle_only)
            g.capture_end()
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            g.replay()               # untimed: instantiation and upload costs
        torch.cuda.synchronize()
        restore()
        return g

    graph = None
    if mode == "graph":
        try:
            graph = capture()
        except Exception as e:  # pragma: no cover
            sys.stderr.write(f"bench.py: graph capture failed ({e!r}); timing plain stream launches\n")
            mode, graph = "stream", None
            torch.cuda.synchronize()
            restore()

    def timed(run):
        """Device time of run() on `stream`, bracketed by barrier + synchronize on both sides."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(stream):
            e0.record()
            run()
            e1.record()
        barrier()
        return e0.elapsed_time(e1)

    # ---- the timed region: K steps, nothing but the path's kernels between the two events -------------
    sampler = ClockSampler(local)
    sampler.start()
    if graph is not None:
        elapsed_ms = timed(graph.replay)
    else:
        elapsed_ms = timed(lambda: [step(W_steps + s) for s in range(K_steps)])
    window = "timed region"
    # results of the timed steps (every step does the same work on identical copies)
    n_commit_h = n_commit.cpu().numpy()
    accepted_h = accepted.cpu().numpy()
    select_h = select.cpu().numpy()
    status_h = status.cpu().numpy()
    sel_len_after = sel_len.cpu().numpy()
    if len(sampler.samples) < 5 and graph is not None:
        # region too short for the sampler: keep the same graph running, untimed, while sampling
        window = "timed region + untimed repeats of the same graph"
        t_end = time.time() + 0.3
        while time.time() < t_end:
            restore()
            with torch.cuda.stream(stream):
                graph.replay()
            torch.cuda.synchronize()
    sampler.stop_flag.set()
    sampler.join(timeout=2)

    # ---- per-kernel times: the same K steps again, (a) with event records around the verify call
    # inside the graph (each record is a graph node of its own and costs a few microseconds of
    # serialisation, so these are upper bounds), (b) without the verify call (difference to the
    # timed region = what verify adds to a step) ------------------------------------------------------
    kt = None
    if not args.no_kernel_events:
        try:
            restore()
            ext = graph is not None
            evs = [[torch.cuda.Event(enable_timing=True, external=ext) for _ in range(3)] for _ in range(K_steps)]
            if graph is not None:
                g_ev = capture(evs)
                t_ev = timed(g_ev.replay)
                restore()
                g_nv = capture(None, with_verify=False)
                restore()
                t_nv = timed(g_nv.replay)
                g_lk = capture(None, lookup_only=True)
                t_lk = timed(g_lk.replay)
                restore()
                g_vo = capture(None, verify_only=True)
                restore()
                t_vo = timed(g_vo.replay)
                g_pr = capture(None, probe_only=True)
                t_pr = timed(g_pr.replay)
                restore()
                g_cy = capture(None, cycle_only=True)
                restore()
                t_cy = timed(g_cy.replay)
            else:
                t_ev = timed(lambda: [step(W_steps + s, evs[s]) for s in range(K_steps)])
                restore()
                t_nv = timed(lambda: [step(W_steps + s, None, False) for s in range(K_steps)])
                t_lk = timed(lambda: [step(W_steps + s, None, False, True) for s in range(K_steps)])
                restore()
                t_vo = timed(lambda: [step(W_steps + s, None, True, False, True) for s in range(K_steps)])
                t_pr = timed(lambda: [step(W_steps + s, probe_only=True) for s in range(K_steps)])
                restore()
                t_cy = timed(lambda: [step(W_steps + s, cycle_only=True) for s in range(K_steps)])
            restore()
            d = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(2)] for e in evs])
            kt = {"lookup_plus_score_select_us": 1e3 * float(d[:, 0].mean()),
                  "verify_commit_us": 1e3 * float(d[:, 1].mean()),
                  "verify_commit_us_median": 1e3 * float(np.median(d[:, 1])),
                  "step_us_with_event_records": 1e3 * t_ev / K_steps,
                  "step_us_without_verify": 1e3 * t_nv / K_steps,
                  "lookup_only_us": 1e3 * t_lk / K_steps,
                  "verify_commit_us_by_difference": 1e3 * (elapsed_ms - t_nv) / K_steps,
                  "verify_commit_us_back_to_back": 1e3 * t_vo / K_steps,
                  "read_probe_us": 1e3 * t_pr / K_steps,
                  "step_us_commit_fused_with_next_lookup": 1e3 * t_cy / K_steps,
                  "note": "event-bracketed times include the serialisation the event records add; "
                          "the headline region has no records in it"}
        except Exception as e:  # pragma: no cover
            sys.stderr.write(f"bench.py: per-kernel events unavailable ({e!r})\n")

    elapsed_ms = max_over_ranks(elapsed_ms, dev)
    steps_per_s = world * K_steps / (elapsed_ms * 1e-3)
    tokens_per_step = int(n_commit_h.sum())
    assert (status_h == 0).all(), "a request reported a capacity or length problem"

    # ---- roofline of the dominant kernel (verify/commit): algorithmic bytes = needed rows x V x elt ----
    verify_bytes = int((sel_len_after.astype(np.int64) + 1).sum()) * w.V * w.elt
    lookup_bytes = int(rq.hist_len.astype(np.int64).sum()) * 4
    roofline = {"bound": "hbm", "kernel": "verify_stream_kernel (+ verify_commit_kernel)", "achieved": None, "peak": peak_gbs, "unit": "GB/s",
                "frac": None, "traffic": NCU_VERIFY_TRAFFIC_BYTES.get(w.name), "peak_kind": peak_kind,
                "algorithmic_bytes_per_launch": verify_bytes}
    roofline_lookup = {"bound": "hbm", "kernel": "lookup_kernel (hvd_lookup alone, back to back in one graph)",
                       "achieved": None, "peak": peak_gbs, "unit": "GB/s", "frac": None, "traffic": None,
                       "peak_kind": peak_kind, "algorithmic_bytes_per_launch": lookup_bytes}
    if kt:
        roofline["achieved"] = verify_bytes / (kt["verify_commit_us_back_to_back"] * 1e-6) / 1e9
        roofline["frac"] = roofline["achieved"] / peak_gbs
        roofline["frac_of_8000_nominal"] = roofline["achieved"] / 8000.0
        roofline["achieved_by_difference"] = verify_bytes / (kt["verify_commit_us_by_difference"] * 1e-6) / 1e9
        roofline["achieved_with_event_records_in_graph"] = verify_bytes / (kt["verify_commit_us"] * 1e-6) / 1e9
        roofline_lookup["achieved"] = lookup_bytes / (kt["lookup_only_us"] * 1e-6) / 1e9
        roofline_lookup["frac"] = roofline_lookup["achieved"] / peak_gbs
        probe_bytes = logits[0].numel() * logits[0].element_size()
        roofline["read_only_kernel"] = {"achieved": probe_bytes / (kt["read_probe_us"] * 1e-6) / 1e9, "unit": "GB/s",
                                        "bytes_per_launch": probe_bytes,
                                        "what": "hvd_read_probe: a plain grid-stride read of the whole logits buffer, "
                                                "timed like the verify call (K launches back to back on the rotating copies)"}
        roofline["frac_of_read_only_kernel"] = roofline["achieved"] / roofline["read_only_kernel"]["achieved"]
        roofline["timing"] = ("CUDA events around a graph of the same K hvd_verify_commit launches back to back "
                              "(both kernels of the call, launch gaps included), on rotating inputs larger than L2")

    # ---- end to end through the host-buffer entry point --------------------------------------------
    e2e = None
    if not args.no_e2e:
        E = max(1, min(args.e2e_steps, K_steps))
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        h_hist, h_off, h_cap = pin(rq.hist), pin(rq.hist_off), pin(rq.hist_cap)
        h_len, h_K, h_pl = pin(rq.hist_len), pin(rq.K), pin(rq.prompt_len)
        h_state = pin(rq.state.view(np.int64).reshape(B, 2))
        h_md, h_ml, h_ro = pin(rq.model_draft), pin(rq.model_len), pin(rq.row_off)
        h_logits = torch.empty(logits0.shape, dtype=logits0.dtype, pin_memory=True)
        h_logits.copy_(logits0)
        hz = lambda *s: torch.zeros(s, dtype=torch.int32).pin_memory()
        o_score = torch.zeros(B, dtype=torch.float32).pin_memory()
        o_sel, o_sd, o_sl, o_acc, o_com, o_nc, o_st = hz(B), hz(B, kc), hz(B), hz(B), hz(B, kc + 1), hz(B), hz(B)
        len0, st0 = h_len.clone(), h_state.clone()

        def host_step():
            h_len.copy_(len0)
            h_state.copy_(st0)
            ctx.hvd_step_host(B=B, n_max=n_max, hist=h_hist, hist_off=h_off, hist_cap=h_cap, hist_len=h_len,
                              K=h_K, prompt_len=h_pl, state=h_state, model_draft=h_md, model_len=h_ml,
                              logits=h_logits, dtype=dtype, V=w.V, row_off=h_ro, k_uniform=0,
                              total_rows=total_rows, score=o_score, select=o_sel, sel_draft=o_sd,
                              sel_len=o_sl, accepted=o_acc, committed=o_com, n_commit=o_nc, status=o_st)

        for _ in range(3):
            host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(E):
            host_step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, dev)
        assert (o_acc.numpy() == accepted_h).all() and (o_nc.numpy() == n_commit_h).all()
        small = B * (8 + 4 * 5 + 16) + (B + 1) * 8 + B * kc * 4
        # of the logits the call copies the rows verification reads (rows 0..sel_len of every request)
        logits_h2d = int((o_sl.numpy().astype(np.int64) + 1).sum()) * w.V * w.elt
        h2d = int(h_hist.numel() * 4 + logits_h2d + small)
        d2h = int(B * 4 * 7 + B * kc * 4 + B * (kc + 1) * 4 + B * 16)
        e2e = {"value": world * E / dt, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": E, "ms_per_step": 1e3 * dt / E, "tokens_per_s": world * E * tokens_per_step / dt,
               "api": "hvd_step_host (pinned host buffers)",
               "logits_bytes_on_host": int(h_logits.numel() * h_logits.element_size()),
               "note": "histories, per-request arrays and the logits rows that verification reads cross the bus "
                       "every step (the rows beyond a request's selected draft are not copied)"}

    # ---- CPU baseline: the oracle, as it stands, on this machine's host cores (rank 0, N = 1) ----------
    cpu_baseline = None
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        from oracle import pipeline as P
        cores = P.host_threads()
        logits_np = W.logits_to_numpy(logits0)
        inp = P.Inputs(w, rq, W1, b1, W2, b2, tau, Wh=Wh, bh=bh, A=A, strict=np.ones(B, bool), logits_np=logits_np)
        times, out = [], None
        t_begin = time.perf_counter()
        while len(times) < 5 or (time.perf_counter() - t_begin < 10.0 and len(times) < 200):
            rq_c = rq.copy()
            t0 = time.perf_counter()
            out = P.step(inp, rq_c, nthreads=cores)
            times.append(time.perf_counter() - t0)
        med = float(np.median(times))
        same = bool((out.vf.accepted == accepted_h).all() and (out.vf.n_commit == n_commit_h).all()
                    and (out.sc.select == select_h).all())
        cpu_baseline = {"value": 1.0 / med, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"the whole {w.name} batch ({B} requests, {total_rows} logits rows), "
                                  f"median of {len(times)} repetitions",
                        "ms_per_step": 1e3 * med, "tokens_per_s": tokens_per_step / med,
                        "agrees_with_gpu_step": same}

    if rank == 0:
        line = {"metric": METRIC, "value": steps_per_s, "unit": UNIT, "n_gpus": world, "steps": K_steps,
                "warmup": W_steps, "ms_per_step": elapsed_ms / K_steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
                "config": workload_config(w, world, {
                    "cold_cache": f"{R} rotating copies of histories+logits ({foot / 2**20:.0f} MiB each, "
                                  f"L2 is 126 MiB); inputs per step exceed L2",
                    "launch": f"{mode}: {K_steps} steps x {4 if args.unfused else 3} kernels in one CUDA graph"
                              if graph is not None else f"stream: {4 if args.unfused else 3} kernel launches per step",
                    "entry_points": "hvd_lookup + hvd_score_select + hvd_verify_commit" if args.unfused
                                    else "hvd_lookup_score_select + hvd_verify_commit",
                    "kernel_events_in_timed_region": False, "tau": tau,
                    "predictor": f"8->{w.hidden}" + (f"->{w.hidden}" if w.hidden_layers == 2 else "") + "->1 fp32"}),
                "tokens_per_s": world * K_steps * tokens_per_step / (elapsed_ms * 1e-3),
                "tokens_per_step": tokens_per_step,
                "mean_accepted": float(accepted_h.mean()), "cache_selected_frac": float(select_h.mean()),
                "kernel_us": kt, "roofline": roofline, "roofline_lookup": roofline_lookup,
                "lookup_algorithmic_bytes": lookup_bytes,
                # the whole step against the same peak: history bytes scanned + logits bytes read, per rank
                "roofline_step": {"bound": "hbm", "algorithmic_bytes_per_step": lookup_bytes + verify_bytes,
                                  "achieved": (lookup_bytes + verify_bytes) / (elapsed_ms / K_steps * 1e-3) / 1e9,
                                  "peak": peak_gbs, "unit": "GB/s", "peak_kind": peak_kind,
                                  "frac": (lookup_bytes + verify_bytes) / (elapsed_ms / K_steps * 1e-3) / 1e9 / peak_gbs},
                "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": (4 if args.unfused else 3) * K_steps,
                "clocks": sampler.summary(window)}
        if kt:
            # the same K steps with hvd_verify_commit_next (commit + next cycle's lookup and selection in one
            # kernel: two launches per step), single rank's figure; the headline keeps the separate entry points
            line["variant_commit_fused_with_next_lookup"] = {
                "value": 1.0 / (kt["step_us_commit_fused_with_next_lookup"] * 1e-6), "unit": UNIT,
                "us_per_step": kt["step_us_commit_fused_with_next_lookup"],
                "entry_points": "hvd_verify_commit_next (after one hvd_lookup_score_select)"}
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
